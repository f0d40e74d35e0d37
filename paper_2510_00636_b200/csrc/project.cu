// Window queries from hidden states (Eq. 5: q = W_Q h before the rotary embedding) on the tcgen05
// tensor cores:  Q[u, j, w, :] = W_Q^j H[u, w, :]  for the W buffered hidden states of unit u and
// every query head j, bf16 x bf16 -> fp32.  Mean and covariance of these rows are W_Q mu_h and
// W_Q Sigma_h W_Q^T exactly, so the statistics kernels take Q in place of the d_model x d_model
// covariance of the hidden states (about Hq*d/W times fewer FLOPs, and no d_model^2 intermediate).
//
// The projection matrix is the large operand (Hq*d x d_model per layer, read once from HBM); the
// hidden-state buffer is small and stays in L2.  A CTA owns 128 rows of W_Q (an N tile) of one unit
// and all of the unit's window rows (up to four M tiles of 128, each with its own accumulator in
// tensor memory), and streams the d_model axis in 64-channel chunks through a TMA ring:
//   warp 0    TMA producer (one lane)
//   warp 1    MMA issuer (one lane); owns the tensor-memory allocation
//   warps 2-5 epilogue: thread <-> accumulator lane <-> window row, fp32 rows to global memory
// Every wait is bounded; a wait that gives up raises the context's status word.
#include "ea_internal.h"
#include "ptx_sm100.cuh"

namespace {

using namespace ptx;

constexpr int kPjThreads = 192;
constexpr int kPjTile = 128;                       // rows per M tile (window) and per N tile (W_Q rows)
constexpr int kPjChunk = kPjTile * 128;            // bytes of one 64-channel chunk of a 128-row tile
constexpr int kPjMaxMTiles = 4;
constexpr int kPjSmemBudget = 200 * 1024;

struct PjParams {
    float* q;                // fp32 [n_units, Hq, W, d]
    int* status;
    int Hq, d, W;
    int n_cols;              // Hq * d
    int k_chunks;            // ceil(d_model / 64)
    int m_tiles;             // ceil(W / 128)
    int stages;
    int units_per_set;
};

__global__ void __launch_bounds__(kPjThreads, 1)
project_kernel(const __grid_constant__ CUtensorMap h_map, const __grid_constant__ CUtensorMap w_map,
               const PjParams p) {
    extern __shared__ uint8_t smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const int stage_bytes = (1 + p.m_tiles) * kPjChunk;
    const uint32_t s_bar = base + (uint32_t)(p.stages * stage_bytes);
    uint8_t* bar_gen = gen_base + p.stages * stage_bytes;
    auto full = [&](int s) { return s_bar + 8u * s; };
    auto empty = [&](int s) { return s_bar + 8u * (8 + s); };
    const uint32_t tmem_full = s_bar + 8u * 16;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * 17);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * 17 + 4);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int n0 = blockIdx.x * kPjTile;
    const int u = blockIdx.y;
    const uint32_t tmem_cols = p.m_tiles <= 1 ? 128u : (p.m_tiles == 2 ? 256u : 512u);

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(full(s), 1);
            mbar_init(empty(s), 1);
        }
        mbar_init(tmem_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&h_map);
        prefetch_tensormap(&w_map);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            bool ok = true;
            int kc = 0;
            for (; ok && kc < p.k_chunks; ++kc) {
                const int s = kc % p.stages;
                const uint32_t fill = (uint32_t)(kc / p.stages);
                ok = mbar_wait(empty(s), (fill & 1) ^ 1, abort_flag);
                if (!ok) break;
                const uint32_t dst = base + (uint32_t)(s * stage_bytes);
                mbar_arrive_expect_tx(full(s), (uint32_t)stage_bytes);
                tma_load_3d(dst, &w_map, full(s), kc * 64, n0, u / p.units_per_set);
                for (int mt = 0; mt < p.m_tiles; ++mt)
                    tma_load_3d(dst + (uint32_t)((1 + mt) * kPjChunk), &h_map, full(s), kc * 64, mt * kPjTile, u);
            }
            if (!ok) {
                // let the copies already in flight land before the CTA's shared memory goes away
                for (int back = 1; back <= p.stages && back <= kc; ++back) {
                    const int c = kc - back;
                    mbar_drain(full(c % p.stages), (uint32_t)(c / p.stages) & 1);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16_m128(kPjTile);
            bool ok = true;
            for (int kc = 0; ok && kc < p.k_chunks; ++kc) {
                const int s = kc % p.stages;
                ok = mbar_wait(full(s), (uint32_t)(kc / p.stages) & 1, abort_flag);
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t s_w = base + (uint32_t)(s * stage_bytes);
                for (int mt = 0; mt < p.m_tiles; ++mt) {
                    const uint32_t s_h = s_w + (uint32_t)((1 + mt) * kPjChunk);
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks)
                        umma_bf16(tmem_base + (uint32_t)(mt * kPjTile), umma_desc_k_sw128(s_h + ks * 32),
                                  umma_desc_k_sw128(s_w + ks * 32), idesc, (kc | ks) ? 1u : 0u);
                }
                umma_commit(empty(s));          // the stage is free once these MMAs have read it
            }
            if (ok) umma_commit(tmem_full);
        }
        __syncwarp();
    } else {
        const int quarter = warp % 4;              // the tensor-memory lanes this warp may read
        bool ok = mbar_wait(tmem_full, 0u, abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (ok) {
            tc_fence_after_sync();
            for (int mt = 0; mt < p.m_tiles; ++mt) {
                const int w = mt * kPjTile + quarter * 32 + lane;
#pragma unroll 1
                for (int cb = 0; cb < kPjTile / 32; ++cb) {
                    uint32_t acc[32];
                    tmem_ld_x32(tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(mt * kPjTile + cb * 32), acc);
                    tmem_ld_wait();
                    const int col = n0 + cb * 32;
                    if (w < p.W && col < p.n_cols) {
                        const int j = col / p.d, c = col % p.d;      // a 32-column block lies inside one head
                        float4* dst = reinterpret_cast<float4*>(p.q + (((size_t)u * p.Hq + j) * p.W + w) * p.d + c);
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            dst[e] = make_float4(__uint_as_float(acc[4 * e]), __uint_as_float(acc[4 * e + 1]),
                                                 __uint_as_float(acc[4 * e + 2]), __uint_as_float(acc[4 * e + 3]));
                    }
                }
            }
        }
    }

    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, tmem_cols);
    }
    if (threadIdx.x == 0 && *abort_flag) *p.status = (int)EA_ERR_DEVICE_TIMEOUT;
}

}  // namespace

bool ea_project_supported(const ea_shape& s, int d_model) {
    return d_model >= 8 && d_model % 8 == 0 && s.window >= 1 && s.window <= kPjMaxMTiles * kPjTile;
}

ea_status ea_launch_project(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* hidden,
                            const __nv_bfloat16* w_q, int d_model, int n_sets, float* q_win, cudaStream_t st) {
    if (!ea_project_supported(s, d_model)) return EA_ERR_UNSUPPORTED;
    PjParams p;
    p.q = q_win;
    p.status = ctx->status_dev;
    p.Hq = s.n_q_heads;
    p.d = s.head_dim;
    p.W = s.window;
    p.n_cols = s.n_q_heads * s.head_dim;
    p.k_chunks = (d_model + 63) / 64;
    p.m_tiles = (s.window + kPjTile - 1) / kPjTile;
    const int stage_bytes = (1 + p.m_tiles) * kPjChunk;
    p.stages = kPjSmemBudget / stage_bytes;
    if (p.stages > 8) p.stages = 8;
    if (p.stages > p.k_chunks) p.stages = p.k_chunks;
    p.units_per_set = s.n_units / n_sets;
    CUtensorMap h_map, w_map;
    if (!ea_tensor_map_bf16_3d(&h_map, hidden, (uint64_t)d_model, (uint64_t)s.window, (uint64_t)s.n_units,
                               (uint64_t)d_model * 2, (uint64_t)s.window * d_model * 2, 64, kPjTile) ||
        !ea_tensor_map_bf16_3d(&w_map, w_q, (uint64_t)d_model, (uint64_t)p.n_cols, (uint64_t)n_sets,
                               (uint64_t)d_model * 2, (uint64_t)p.n_cols * d_model * 2, 64, kPjTile))
        return EA_ERR_CUDA;
    const int smem = p.stages * stage_bytes + 1024 + 256;
    EA_CUDA_TRY(cudaFuncSetAttribute(project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
    const dim3 grid((unsigned)((p.n_cols + kPjTile - 1) / kPjTile), (unsigned)s.n_units);
    if (grid.y > 65535u) return EA_ERR_UNSUPPORTED;
    project_kernel<<<grid, kPjThreads, smem, st>>>(h_map, w_map, p);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}
