// Log-scores s_{h,i} = mu_bar_h.k_i/sqrt(d) + k_i^T Sigma_bar_h k_i/(2d) (Eq. 7) on the
// tcgen05 tensor cores.
//
// The dense part is the product K . B^T of a tile of 128 cached keys with a bf16 image B of
// the covariance; the row-wise quadratic form is finished in the epilogue:
//     D[i, c]  = sum_a K[i, a] B[c, a]                      (tcgen05.mma, fp32 in tensor memory)
//     s_{h,i}  = sum_c k_{i,c} ( D[i, c]/(2d) + mu_bar_c/sqrt(d) + Sigma_bar_cc k_{i,c}/(2d) )
// B carries the off-diagonal of Sigma_bar at twice bf16 precision for the price of one bf16
// matrix: the quadratic form only sees B[c,a] + B[a,c], so for a < c the entry B[c,a] holds
// bf16(2 Sigma_ac) and the mirrored entry B[a,c] holds the bf16 rounding of what that left over.
// The diagonal stays out of B and enters in fp32 in the epilogue together with the linear term.
//
// One CTA keeps the image of `hpc` query heads of one KV head resident in shared memory
// (hpc * d = 256 accumulator columns at most) and streams key tiles through a TMA ring:
//   warp 0    TMA producer (one lane): covariance image (bulk copy) and key tiles (tiled, 128B swizzle)
//   warp 1    MMA issuer (one lane); owns the tensor-memory allocation
//   warps 2-5 epilogue: thread <-> accumulator lane <-> key; reads its key row from the staged tile
// Tensor memory holds two accumulator stages so the epilogue of one tile overlaps the MMAs of
// the next.  Every wait is bounded; a wait that gives up raises the context's status word.
#include "ea_internal.h"
#include "ptx_sm100.cuh"

namespace {

using namespace ptx;

constexpr int kTileKeys = 128;
constexpr int kEpiWarps = 4;
constexpr int kMmaThreads = 32 * (2 + kEpiWarps);
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;          // columns of one accumulator stage

template <int D>
struct Geo {
    static constexpr int HPC = 256 / D;                  // query heads per CTA pass (1, 2 or 4)
    static constexpr int KCH = D / 64;                   // 64-channel (128-byte) chunks per row
    static constexpr int CHUNK_A = kTileKeys * 128;      // bytes of one chunk of a key tile
    static constexpr int STAGE = KCH * CHUNK_A;          // bytes of one key tile
    static constexpr int IMG_ROWS = HPC * D;             // rows (accumulator columns) of the image
    static constexpr int CHUNK_B = IMG_ROWS * 128;       // bytes of one chunk of the image
    static constexpr int IMG = KCH * CHUNK_B;            // bytes of the image of one head subset
    static constexpr int STAGES = 4;
    static constexpr int VEC = HPC * D * 2 * sizeof(float);   // mu' and diagonal vectors
    static constexpr int SMEM = IMG + STAGES * STAGE + VEC + 256 + 1024;
};

struct MmaParams {
    const float* vec;        // fp32 [U*Hq][2][D]: mu_bar/sqrt(d), diag(Sigma_bar)/(2d)
    const uint8_t* image;    // bf16 images, Geo::IMG bytes per (unit, kv head, head subset)
    float* logits;           // fp32 [U, Hq, n]
    int* status;             // device-visible status word
    int Hq, Hkv, n;
    int n_subsets;           // head subsets per KV head
    int n_tiles;             // key tiles per head
    int chunk_tiles;         // tiles per work item
    int n_chunks;            // work items per (head subset)
    long long n_items;
};

// ------------------------------------------------------------------------------------------
// Covariance image and epilogue vectors.  One CTA per query head.
template <int D>
__global__ void __launch_bounds__(256)
sigma_image_kernel(const float* __restrict__ mu_bar, const float* __restrict__ sigma_bar, int Hq, int Hkv,
                   uint8_t* __restrict__ image, float* __restrict__ vec) {
    using G = Geo<D>;
    const int uh = blockIdx.x;
    const int u = uh / Hq, h = uh % Hq;
    const int Gq = Hq / Hkv;
    const int g = h / Gq, hg = h % Gq;
    const int n_subsets = (Gq + G::HPC - 1) / G::HPC;
    const int hs = hg / G::HPC, j = hg % G::HPC;
    const float* S = sigma_bar + (size_t)uh * D * D;
    uint8_t* img = image + ((size_t)(u * Hkv + g) * n_subsets + hs) * G::IMG;

    // one 16-byte unit (8 consecutive a) of one row c per thread step
    for (int e = threadIdx.x; e < D * (D / 8); e += blockDim.x) {
        const int c = e / (D / 8), a0 = (e % (D / 8)) * 8;
        uint32_t w[4];
#pragma unroll
        for (int p = 0; p < 4; ++p) {
            uint32_t half[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int a = a0 + 2 * p + q;
                float val = 0.f;
                if (a != c) {
                    const float two_s = S[(size_t)c * D + a] + S[(size_t)a * D + c];
                    const float hi = __bfloat162float(__float2bfloat16_rn(two_s));
                    val = a < c ? hi : two_s - hi;
                }
                half[q] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(val));
            }
            w[p] = half[0] | (half[1] << 16);
        }
        const int row = j * D + c;
        const int kc = a0 / 64, unit = (a0 % 64) / 8;
        uint4* dst = reinterpret_cast<uint4*>(img + (size_t)kc * G::CHUNK_B + (size_t)row * 128 +
                                              ((unit ^ (row & 7)) << 4));
        *dst = make_uint4(w[0], w[1], w[2], w[3]);
    }
    const float inv_sqrt_d = rsqrtf((float)D), inv_2d = 0.5f / (float)D;
    for (int c = threadIdx.x; c < D; c += blockDim.x) {
        vec[((size_t)uh * 2 + 0) * D + c] = mu_bar[(size_t)uh * D + c] * inv_sqrt_d;
        vec[((size_t)uh * 2 + 1) * D + c] = S[(size_t)c * D + c] * inv_2d;
    }
}

// ------------------------------------------------------------------------------------------
struct Item {
    int ug, hs, tile0, tile1, hpc;
};

__device__ __forceinline__ Item decode_item(long long item, const MmaParams& p, int hpc_max) {
    Item it;
    it.hs = (int)(item % p.n_subsets);
    const long long r = item / p.n_subsets;
    const int chunk = (int)(r % p.n_chunks);
    it.ug = (int)(r / p.n_chunks);
    it.tile0 = chunk * p.chunk_tiles;
    it.tile1 = min(p.n_tiles, it.tile0 + p.chunk_tiles);
    const int Gq = p.Hq / p.Hkv;
    it.hpc = min(hpc_max, Gq - it.hs * hpc_max);
    return it;
}

template <int D>
__global__ void __launch_bounds__(kMmaThreads, 1)
logits_mma_kernel(const __grid_constant__ CUtensorMap k_map, const MmaParams p) {
    using G = Geo<D>;
    extern __shared__ uint8_t smem_raw[];
    // carve shared memory: 1024-byte aligned operand tiles first
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t s_img = base;
    const uint32_t s_k = s_img + G::IMG;
    const uint32_t s_vec = s_k + G::STAGES * G::STAGE;
    const float* vec_gen = reinterpret_cast<const float*>(gen_base + G::IMG + G::STAGES * G::STAGE);
    const uint32_t s_bar = s_vec + G::VEC;
    uint8_t* bar_gen = gen_base + G::IMG + G::STAGES * G::STAGE + G::VEC;
    // barriers: full_k[S], empty_k[S], tmem_full[2], tmem_empty[2], img_full
    auto full_k = [&](int s) { return s_bar + 8u * s; };
    auto empty_k = [&](int s) { return s_bar + 8u * (G::STAGES + s); };
    auto tmem_full = [&](int a) { return s_bar + 8u * (2 * G::STAGES + a); };
    auto tmem_empty = [&](int a) { return s_bar + 8u * (2 * G::STAGES + 2 + a); };
    const uint32_t img_full = s_bar + 8u * (2 * G::STAGES + 4);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * (2 * G::STAGES + 5));
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * (2 * G::STAGES + 5) + 4);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;

    if (threadIdx.x == 0) {
        for (int s = 0; s < G::STAGES; ++s) {
            mbar_init(full_k(s), 1);
            mbar_init(empty_k(s), kEpiWarps);
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(tmem_full(a), 1);
            mbar_init(tmem_empty(a), kEpiWarps);
        }
        mbar_init(img_full, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&k_map);
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const long long first = blockIdx.x, stride = gridDim.x;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            int fills[G::STAGES];
#pragma unroll
            for (int s = 0; s < G::STAGES; ++s) fills[s] = 0;
            long long tile_no = 0;
            long long cur_img = -1;
            bool ok = true;
            for (long long item = first; ok && item < p.n_items; item += stride) {
                const Item it = decode_item(item, p, G::HPC);
                const long long img_id = (long long)it.ug * p.n_subsets + it.hs;
                if (img_id != cur_img) {
                    // every tile that used the resident image must have left the epilogue
#pragma unroll
                    for (int s = 0; s < G::STAGES; ++s)
                        if (ok && fills[s] > 0) ok = mbar_wait(empty_k(s), (fills[s] - 1) & 1, abort_flag);
                    if (!ok) break;
                    const int rows = it.hpc * D;
                    const int u = it.ug / p.Hkv, g = it.ug % p.Hkv;
                    const int h0 = g * (p.Hq / p.Hkv) + it.hs * G::HPC;
                    const uint32_t vec_bytes = (uint32_t)(it.hpc * 2 * D * sizeof(float));
                    mbar_arrive_expect_tx(img_full, (uint32_t)(G::KCH * rows * 128) + vec_bytes);
                    const uint8_t* src = p.image + (size_t)img_id * G::IMG;
                    for (int kc = 0; kc < G::KCH; ++kc)
                        bulk_load(s_img + kc * G::CHUNK_B, src + (size_t)kc * G::CHUNK_B, rows * 128, img_full);
                    bulk_load(s_vec, p.vec + ((size_t)u * p.Hq + h0) * 2 * D, vec_bytes, img_full);
                    cur_img = img_id;
                }
                for (int t = it.tile0; ok && t < it.tile1; ++t, ++tile_no) {
                    const int s = (int)(tile_no % G::STAGES);
                    ok = mbar_wait(empty_k(s), (fills[s] & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    mbar_arrive_expect_tx(full_k(s), G::STAGE);
                    for (int kc = 0; kc < G::KCH; ++kc)
                        tma_load_3d(s_k + s * G::STAGE + kc * G::CHUNK_A, &k_map, full_k(s), kc * 64,
                                    t * kTileKeys, it.ug);
                    ++fills[s];
                }
            }
            if (!ok) {
                // let the copies already in flight land before the CTA's shared memory goes away
#pragma unroll
                for (int s = 0; s < G::STAGES; ++s)
                    if (fills[s] > 0) mbar_wait(full_k(s), (fills[s] - 1) & 1, abort_flag);
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            long long tile_no = 0, cur_img = -1;
            int img_loads = 0;
            bool ok = true;
            for (long long item = first; ok && item < p.n_items; item += stride) {
                const Item it = decode_item(item, p, G::HPC);
                const long long img_id = (long long)it.ug * p.n_subsets + it.hs;
                if (img_id != cur_img) {
                    ok = mbar_wait(img_full, img_loads & 1, abort_flag);
                    if (!ok) break;
                    ++img_loads;
                    cur_img = img_id;
                }
                const uint32_t idesc = umma_idesc_bf16_m128((uint32_t)(it.hpc * D));
                for (int t = it.tile0; ok && t < it.tile1; ++t, ++tile_no) {
                    const int s = (int)(tile_no % G::STAGES);
                    const int a = (int)(tile_no & 1);
                    const uint32_t use = (uint32_t)(tile_no >> 1);
                    ok = mbar_wait(full_k(s), (uint32_t)((tile_no / G::STAGES) & 1), abort_flag) &&
                         mbar_wait(tmem_empty(a), (use & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(a * kAccCols);
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t off = (uint32_t)((ks % 4) * 32);
                        const uint64_t da = umma_desc_k_sw128(s_k + s * G::STAGE + (ks / 4) * G::CHUNK_A + off);
                        const uint64_t db = umma_desc_k_sw128(s_img + (ks / 4) * G::CHUNK_B + off);
                        umma_bf16(d_tmem, da, db, idesc, ks > 0 ? 1u : 0u);
                    }
                    umma_commit(tmem_full(a));
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ epilogue
        const int quarter = warp % 4;              // the TMEM lanes this warp may read
        const int row = quarter * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const float inv_2d = 0.5f / (float)D;
        long long tile_no = 0, cur_img = -1;
        int img_loads = 0;
        bool ok = true;
        for (long long item = first; ok && item < p.n_items; item += stride) {
            const Item it = decode_item(item, p, G::HPC);
            const long long img_id = (long long)it.ug * p.n_subsets + it.hs;
            if (img_id != cur_img) {
                ok = __all_sync(0xffffffffu, mbar_wait(img_full, img_loads & 1, abort_flag));
                if (!ok) break;
                ++img_loads;
                cur_img = img_id;
            }
            const int u = it.ug / p.Hkv, g = it.ug % p.Hkv;
            const int h0 = g * (p.Hq / p.Hkv) + it.hs * G::HPC;
            for (int t = it.tile0; ok && t < it.tile1; ++t, ++tile_no) {
                const int s = (int)(tile_no % G::STAGES);
                const int a = (int)(tile_no & 1);
                ok = __all_sync(0xffffffffu, mbar_wait(tmem_full(a), (uint32_t)((tile_no >> 1) & 1), abort_flag));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t k_row = s_k + s * G::STAGE + row * 128;
                float2 acc[G::HPC];
#pragma unroll
                for (int j = 0; j < G::HPC; ++j) acc[j] = make_float2(0.f, 0.f);
#pragma unroll
                for (int cb = 0; cb < D / 32; ++cb) {
                    const int c0 = cb * 32;
                    float2 kf[16];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int unit = (c0 % 64) / 8 + q;
                        const uint4 w = lds128(k_row + (c0 / 64) * G::CHUNK_A + ((unit ^ (row & 7)) << 4));
                        const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            kf[q * 4 + e] = make_float2(__uint_as_float(ww[e] << 16),
                                                        __uint_as_float(ww[e] & 0xffff0000u));
                    }
#pragma unroll
                    for (int j = 0; j < G::HPC; ++j) {
                        if (j < it.hpc) {
                            uint32_t dv[32];
                            tmem_ld_x32(t_lane + (uint32_t)(a * kAccCols + j * D + c0), dv);
                            tmem_ld_wait();
                            const float4* mu4 = reinterpret_cast<const float4*>(vec_gen + (j * 2 + 0) * D + c0);
                            const float4* dg4 = reinterpret_cast<const float4*>(vec_gen + (j * 2 + 1) * D + c0);
#pragma unroll
                            for (int q = 0; q < 8; ++q) {
                                const float4 m = mu4[q], dg = dg4[q];
                                const float2 k0 = kf[2 * q], k1 = kf[2 * q + 1];
                                float2 t0 = fma2(make_float2(dg.x, dg.y), k0, make_float2(m.x, m.y));
                                float2 t1 = fma2(make_float2(dg.z, dg.w), k1, make_float2(m.z, m.w));
                                t0 = fma2(make_float2(__uint_as_float(dv[4 * q]), __uint_as_float(dv[4 * q + 1])),
                                          make_float2(inv_2d, inv_2d), t0);
                                t1 = fma2(make_float2(__uint_as_float(dv[4 * q + 2]), __uint_as_float(dv[4 * q + 3])),
                                          make_float2(inv_2d, inv_2d), t1);
                                acc[j] = fma2(k0, t0, acc[j]);
                                acc[j] = fma2(k1, t1, acc[j]);
                            }
                        }
                    }
                }
                // the accumulator stage and the key tile are free again
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(tmem_empty(a));
                    mbar_arrive(empty_k(s));
                }
                const int key = t * kTileKeys + row;
                if (key < p.n) {
#pragma unroll
                    for (int j = 0; j < G::HPC; ++j)
                        if (j < it.hpc)
                            p.logits[((size_t)u * p.Hq + h0 + j) * (size_t)p.n + key] = acc[j].x + acc[j].y;
                }
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after_sync();
        tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && *abort_flag) *p.status = (int)EA_ERR_DEVICE_TIMEOUT;
}

// ------------------------------------------------------------------------------------------
typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                    const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                    CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                    CUtensorMapFloatOOBfill);

encode_tiled_fn get_encode_tiled() {
    static encode_tiled_fn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &res) == cudaSuccess &&
            res == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(ptr);
        else
            cudaGetLastError();
    }
    return fn;
}

// K as a rank-3 tensor (d, n, unit*kv_head); one box is 64 channels x 128 keys, 128-byte swizzle.
// Rows past n read as zero.
bool make_k_map(CUtensorMap* map, const __nv_bfloat16* k, int d, int n, long long heads) {
    encode_tiled_fn enc = get_encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)n, (cuuint64_t)heads};
    const cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)n * d * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)kTileKeys, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(k), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

template <int D>
ea_status launch_mma(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* k, const float* mu_bar,
                     const float* sigma_bar, uint8_t* image, float* vec, float* logits, cudaStream_t st) {
    using G = Geo<D>;
    const int Gq = s.n_q_heads / s.n_kv_heads;
    MmaParams p;
    p.vec = vec;
    p.image = image;
    p.logits = logits;
    p.status = ctx->status_dev;
    p.Hq = s.n_q_heads;
    p.Hkv = s.n_kv_heads;
    p.n = s.n_keys;
    p.n_subsets = (Gq + G::HPC - 1) / G::HPC;
    p.n_tiles = (s.n_keys + kTileKeys - 1) / kTileKeys;
    // Work items: enough of them to balance the SMs, long enough to amortise the image load.
    const long long combos = (long long)s.n_units * s.n_kv_heads * p.n_subsets;
    int chunk = p.n_tiles;
    const long long want_items = 6LL * ctx->sm_count;
    while (chunk > 16 && combos * ((p.n_tiles + chunk - 1) / chunk) < want_items) chunk = (chunk + 1) / 2;
    p.chunk_tiles = chunk;
    p.n_chunks = (p.n_tiles + chunk - 1) / chunk;
    p.n_items = combos * p.n_chunks;

    CUtensorMap k_map;
    if (!make_k_map(&k_map, k, D, s.n_keys, (long long)s.n_units * s.n_kv_heads)) return EA_ERR_CUDA;

    sigma_image_kernel<D><<<s.n_units * s.n_q_heads, 256, 0, st>>>(mu_bar, sigma_bar, s.n_q_heads, s.n_kv_heads,
                                                                 image, vec);
    if (cudaFuncSetAttribute(logits_mma_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM) !=
        cudaSuccess)
        return EA_ERR_CUDA;
    const unsigned grid = (unsigned)(p.n_items < ctx->sm_count ? p.n_items : ctx->sm_count);
    ea_count_launches(ctx, 2);
    cudaEvent_t stop = ea_profile_mark_start(ctx, st);
    logits_mma_kernel<D><<<grid, kMmaThreads, G::SMEM, st>>>(k_map, p);
    ea_profile_mark_stop(ctx, stop, st);
    return cudaGetLastError() == cudaSuccess ? EA_OK : EA_ERR_CUDA;
}

}  // namespace

bool ea_mma_path_supported(const ea_shape& s) {
    return (s.head_dim == 64 || s.head_dim == 128) && s.n_keys >= kTileKeys;
}

size_t ea_mma_image_bytes(const ea_shape& s) {
    const int Gq = s.n_q_heads / s.n_kv_heads;
    const int hpc = 256 / s.head_dim;
    const size_t subsets = (size_t)((Gq + hpc - 1) / hpc);
    return (size_t)s.n_units * s.n_kv_heads * subsets * hpc * s.head_dim * s.head_dim * 2;
}

size_t ea_mma_vec_bytes(const ea_shape& s) {
    return (size_t)s.n_units * s.n_q_heads * 2 * s.head_dim * sizeof(float);
}

ea_status ea_launch_logits_mma(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* k,
                               const float* mu_bar, const float* sigma_bar, void* image, float* vec,
                               float* logits, cudaStream_t st) {
    switch (s.head_dim) {
        case 64:
            return launch_mma<64>(ctx, s, k, mu_bar, sigma_bar, static_cast<uint8_t*>(image), vec, logits, st);
        case 128:
            return launch_mma<128>(ctx, s, k, mu_bar, sigma_bar, static_cast<uint8_t*>(image), vec, logits, st);
        default:
            return EA_ERR_UNSUPPORTED;
    }
}
