// Softmax over positions, GQA reduction and value-norm weighting
// (Eq. 8 and Eq. 9 of the paper with ||v|| in place of ||W_o v||).
//
// lse_kernel: one CTA per softmax row, max-subtracted log-sum-exp with a fixed
// reduction order (bitwise reproducible).
// finalize_kernel: one warp per 32 consecutive keys of a KV head.  The warp
// streams the 32 value rows with 128-bit loads (sum of squares in fp32,
// shuffle-reduced), then lane r finishes key r: coalesced log-score loads,
// exp(s - lse) per query head of the group, (a + eps) * ||v||.
#include "ea_internal.h"
#include "ptx_sm100.cuh"

namespace {

constexpr int kLseThreads = 1024;

__device__ __forceinline__ float block_reduce(float v, bool is_max, float* scratch) {
    const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        float o = __shfl_xor_sync(0xffffffffu, v, off);
        v = is_max ? fmaxf(v, o) : v + o;
    }
    __syncthreads();
    if (lane == 0) scratch[warp] = v;
    __syncthreads();
    if (warp == 0) {
        v = scratch[lane];   // kLseThreads / 32 == 32 partials
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) {
            float o = __shfl_xor_sync(0xffffffffu, v, off);
            v = is_max ? fmaxf(v, o) : v + o;
        }
        if (lane == 0) scratch[0] = v;
    }
    __syncthreads();
    return scratch[0];
}

// Row r of the softmax is the mean over `g_avg` consecutive log-score rows
// (g_avg = 1: every query head has its own softmax).
__global__ void __launch_bounds__(kLseThreads)
lse_kernel(const float* __restrict__ logits, int n, int g_avg, float* __restrict__ lse) {
    __shared__ float scratch[32];
    const float* base = logits + (size_t)blockIdx.x * g_avg * n;
    const float inv_g = 1.0f / (float)g_avg;
    float mx = -INFINITY;
    for (int i = threadIdx.x; i < n; i += kLseThreads) {
        float x = 0.f;
        for (int j = 0; j < g_avg; ++j) x += base[(size_t)j * n + i];
        mx = fmaxf(mx, x * inv_g);
    }
    mx = block_reduce(mx, true, scratch);
    float sum = 0.f;
    for (int i = threadIdx.x; i < n; i += kLseThreads) {
        float x = 0.f;
        for (int j = 0; j < g_avg; ++j) x += base[(size_t)j * n + i];
        sum += expf(x * inv_g - mx);
    }
    sum = block_reduce(sum, false, scratch);
    if (threadIdx.x == 0) lse[blockIdx.x] = mx + logf(sum);
}

constexpr int kFinThreads = 256;

template <int D>
__global__ void __launch_bounds__(kFinThreads)
finalize_kernel(const float* __restrict__ logits, const float* __restrict__ lse,
                const __nv_bfloat16* __restrict__ v, int Hq, int Hkv, int n, int cap, int group_mode,
                float epsilon, float* __restrict__ scores) {
    constexpr int LPR = D / 8;          // lanes per value row (one uint4 = 8 bf16 each)
    constexpr int RPS = 32 / LPR;       // rows per load step
    constexpr int STEPS = 32 / RPS;
    const int G = Hq / Hkv;
    const int ug = blockIdx.y;
    const int u = ug / Hkv, g = ug % Hkv;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int key0 = (blockIdx.x * (kFinThreads / 32) + warp) * 32;
    if (key0 >= n) return;

    const uint4* vrow = reinterpret_cast<const uint4*>(v + ((size_t)ug * cap + key0) * D);
    float my_sumsq = 0.f;
#pragma unroll 4
    for (int t = 0; t < STEPS; ++t) {
        const int r = t * RPS + lane / LPR;
        float ss = 0.f;
        if (key0 + r < n) {
            const uint4 x = __ldg(vrow + (size_t)r * LPR + lane % LPR);
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float lo = __uint_as_float(w[q] << 16);
                const float hi = __uint_as_float(w[q] & 0xffff0000u);
                ss = fmaf(lo, lo, ss);
                ss = fmaf(hi, hi, ss);
            }
        }
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        // lane L owns key L: its row was summed in step L / RPS by lane group L % RPS
        const float mine = __shfl_sync(0xffffffffu, ss, (lane % RPS) * LPR);
        if (t == lane / RPS) my_sumsq = mine;
    }

    const int key = key0 + lane;
    if (key >= n) return;
    float a;
    if (group_mode == EA_GROUP_MEAN_LOGIT) {
        float x = 0.f;
        for (int j = 0; j < G; ++j) x += logits[((size_t)u * Hq + (size_t)g * G + j) * n + key];
        a = expf(x * (1.0f / (float)G) - lse[ug]);
    } else {
        a = 0.f;
        for (int j = 0; j < G; ++j) {
            const size_t uh = (size_t)u * Hq + (size_t)g * G + j;
            a += expf(logits[uh * n + key] - lse[uh]);
        }
        if (group_mode == EA_GROUP_MEAN_PROB) a *= 1.0f / (float)G;
    }
    scores[(size_t)ug * n + key] = (a + epsilon) * sqrtf(my_sumsq);
}


// ------------------------------------------------------------------------------------------
// Value norms on a few SMs (Eq. 9's ||v||, the part of the weighting that does not depend on the
// log-scores), so that the pass over V can run beside the tensor-bound log-score kernel instead of
// after it.  A persistent CTA per SM streams its contiguous share of the value rows through shared
// memory with bulk copies (cp.async.bulk: the copy engine keeps about 190 KiB in flight per SM,
// which register-fed loads cannot).  Every warp serves itself: it owns three 4 KiB slots, waits for
// a slot's copy, takes the rows into registers, starts the copy of its next chunk into the same slot
// and only then reduces; no warp ever waits for another one, because each such hand-over costs
// more than the arithmetic of a chunk.
//   lane = (row of a group of four, eighth of the row); the eight lanes of a row read consecutive
//   16-byte pieces (conflict-free), sum squares in fp32 and meet by shuffles; the norms of a chunk
//   leave as one contiguous run.
constexpr int kVnChunk = 4096;             // bytes per bulk copy
constexpr int kVnSlots = 3;                // slots per warp
constexpr int kVnWarps = 16;
constexpr int kVnThreads = 32 * kVnWarps;
constexpr int kVnSmem = kVnWarps * kVnSlots * kVnChunk;

template <int D>
__global__ void __launch_bounds__(kVnThreads, 1)
vnorm_stream_kernel(const __nv_bfloat16* __restrict__ v, long long n_rows, float* __restrict__ vnorm,
                    int* status) {
    constexpr int ROW_BYTES = 2 * D;
    constexpr int CR = kVnChunk / ROW_BYTES;           // rows per chunk (8, 16 or 32)
    constexpr int PPL = D / 64;                        // 16-byte pieces per lane and row (8 lanes per row)
    constexpr int NG = CR / 4;                         // groups of four rows per chunk
    extern __shared__ __align__(1024) uint8_t vn_smem[];
    __shared__ __align__(8) unsigned long long bars[kVnWarps][kVnSlots];
    __shared__ float norms[kVnWarps][CR];
    __shared__ int abort_flag;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    if (threadIdx.x == 0) {
        for (int w = 0; w < kVnWarps; ++w)
            for (int s = 0; s < kVnSlots; ++s) ptx::mbar_init(ptx::smem_u32(&bars[w][s]), 1);
        abort_flag = 0;
        ptx::fence_mbar_init();
    }
    __syncthreads();
    // this CTA's chunks: a contiguous range; chunk c of it belongs to warp c % kVnWarps
    const long long n_chunks = (n_rows + CR - 1) / CR;
    const long long per = (n_chunks + gridDim.x - 1) / gridDim.x;
    const long long c0 = per * blockIdx.x;
    const long long c1 = c0 + per < n_chunks ? c0 + per : n_chunks;
    const long long mine = c1 - c0 > warp ? (c1 - c0 - warp + kVnWarps - 1) / kVnWarps : 0;   // chunks of this warp
    const uint32_t s_warp = ptx::smem_u32(vn_smem) + (uint32_t)(warp * kVnSlots * kVnChunk);
    auto bar = [&](int s) { return ptx::smem_u32(&bars[warp][s]); };
    auto issue = [&](long long k) {                    // lane 0: start the copy of this warp's k-th chunk
        const long long row0 = (c0 + warp + k * kVnWarps) * CR;
        const long long rows = n_rows - row0 < CR ? n_rows - row0 : CR;
        const uint32_t bytes = (uint32_t)(rows * ROW_BYTES);
        const int s = (int)(k % kVnSlots);
        ptx::mbar_arrive_expect_tx(bar(s), bytes);
        ptx::bulk_load(s_warp + (uint32_t)(s * kVnChunk), reinterpret_cast<const uint8_t*>(v) + row0 * ROW_BYTES, bytes,
                       bar(s));
    };
    if (lane == 0)
        for (long long k = 0; k < kVnSlots && k < mine; ++k) issue(k);
    const int rr = lane / 8, q = lane % 8;
    long long k = 0;
    bool ok = true;
    for (; k < mine; ++k) {
        const int s = (int)(k % kVnSlots);
        ok = ptx::mbar_wait(bar(s), (uint32_t)(k / kVnSlots) & 1, &abort_flag);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        const uint32_t s_rows = s_warp + (uint32_t)(s * kVnChunk);
        // (rows past the end read whatever the slot held and are not stored)
        uint4 x[NG][PPL];
#pragma unroll
        for (int g = 0; g < NG; ++g)
#pragma unroll
            for (int e = 0; e < PPL; ++e)
                x[g][e] = ptx::lds128(s_rows + (uint32_t)((4 * g + rr) * ROW_BYTES + (e * 8 + q) * 16));
        float ss[NG];
#pragma unroll
        for (int g = 0; g < NG; ++g) {
            float2 acc[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
            for (int e = 0; e < PPL; ++e) {
                const uint32_t w[4] = {x[g][e].x, x[g][e].y, x[g][e].z, x[g][e].w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const float2 u = make_float2(__uint_as_float(w[c] << 16), __uint_as_float(w[c] & 0xffff0000u));
                    acc[c & 1] = ptx::fma2(u, u, acc[c & 1]);
                }
            }
            ss[g] = (acc[0].x + acc[1].x) + (acc[0].y + acc[1].y);
        }
        // every lane has consumed its pieces: the slot can take this warp's chunk k + kVnSlots
        __syncwarp();
        if (lane == 0 && k + kVnSlots < mine) {
            ptx::fence_proxy_async_smem();             // the reads above are ordered before the copy engine's writes
            issue(k + kVnSlots);
        }
#pragma unroll
        for (int off = 4; off > 0; off >>= 1)
#pragma unroll
            for (int g = 0; g < NG; ++g) ss[g] += __shfl_xor_sync(0xffffffffu, ss[g], off);
        if (q == 0) {
#pragma unroll
            for (int g = 0; g < NG; ++g) norms[warp][4 * g + rr] = sqrtf(ss[g]);
        }
        __syncwarp();
        const long long row0 = (c0 + warp + k * kVnWarps) * CR;
#pragma unroll
        for (int r = lane; r < CR; r += 32)
            if (row0 + r < n_rows) vnorm[row0 + r] = norms[warp][r];
        __syncwarp();
    }
    if (!ok && lane == 0) {
        // let this warp's copies already in flight land before the shared memory goes away
        for (long long j = k; j < k + kVnSlots && j < mine; ++j)
            ptx::mbar_drain(bar((int)(j % kVnSlots)), (uint32_t)(j / kVnSlots) & 1);
    }
    __syncthreads();
    if (threadIdx.x == 0 && abort_flag) *status = (int)EA_ERR_DEVICE_TIMEOUT;
}

// score = (group reduction of the attention + eps) * ||v|| with the norms already computed; one thread per key.
__global__ void __launch_bounds__(256)
weight_kernel(const float* __restrict__ logits, const float* __restrict__ lse, const float* __restrict__ vnorm,
              int vn_stride, int Hq, int Hkv, int n, int group_mode, float epsilon, float* __restrict__ scores) {
    const int G = Hq / Hkv;
    const int ug = blockIdx.y;
    const int u = ug / Hkv, g = ug % Hkv;
    const int key = blockIdx.x * blockDim.x + threadIdx.x;
    if (key >= n) return;
    float a;
    if (group_mode == EA_GROUP_MEAN_LOGIT) {
        float x = 0.f;
        for (int j = 0; j < G; ++j) x += logits[((size_t)u * Hq + (size_t)g * G + j) * n + key];
        a = expf(x * (1.0f / (float)G) - lse[ug]);
    } else {
        a = 0.f;
        for (int j = 0; j < G; ++j) {
            const size_t uh = (size_t)u * Hq + (size_t)g * G + j;
            a += expf(logits[uh * n + key] - lse[uh]);
        }
        if (group_mode == EA_GROUP_MEAN_PROB) a *= 1.0f / (float)G;
    }
    scores[(size_t)ug * n + key] = (a + epsilon) * vnorm[(size_t)ug * vn_stride + key];
}

// ||v|| of a range of rows of every head: lane groups of D / 8 lanes read one row each (128-bit loads), the
// partial sums of squares meet by shuffles, the group's first lane stores the norm.
template <int D>
__global__ void __launch_bounds__(256)
vnorm_rows_kernel(const __nv_bfloat16* __restrict__ v, int cap, int first_row, int n_rows, long long total_rows,
                  float* __restrict__ v_norm) {
    constexpr int LPR = D / 8;                     // lanes per row
    const long long stride = (long long)gridDim.x * blockDim.x / LPR;
    const int lane = threadIdx.x % 32, piece = lane % LPR;
    // the loop bound is the warp's, so that every lane takes part in the shuffles
    for (long long r0 = ((long long)blockIdx.x * blockDim.x + (threadIdx.x - lane)) / LPR; r0 < total_rows; r0 += stride) {
        const long long r = r0 + lane / LPR;
        const bool valid = r < total_rows;
        const long long row = valid ? (r / n_rows) * cap + first_row + r % n_rows : 0;
        float ss = 0.f;
        if (valid) {
            const uint4 x = __ldg(reinterpret_cast<const uint4*>(v + row * D) + piece);
            const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float a = __uint_as_float(w[q] << 16), b = __uint_as_float(w[q] & 0xffff0000u);
                ss = fmaf(a, a, ss);
                ss = fmaf(b, b, ss);
            }
        }
#pragma unroll
        for (int off = LPR / 2; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        if (valid && piece == 0) v_norm[row] = sqrtf(ss);
    }
}

// score = group reduction of (a_hat_h + eps) * sqrt(wo_norm2_h) over the query heads of the KV head
// (Eq. 9 with ||W_o v||); one thread per key.
__global__ void __launch_bounds__(256)
finalize_wo_kernel(const float* __restrict__ logits, const float* __restrict__ lse,
                   const float* __restrict__ wo_norm2, int Hq, int Hkv, int n, int group_mode, float epsilon,
                   float* __restrict__ scores) {
    const int G = Hq / Hkv;
    const int ug = blockIdx.y;
    const int u = ug / Hkv, g = ug % Hkv;
    const int key = blockIdx.x * blockDim.x + threadIdx.x;
    if (key >= n) return;
    float acc = 0.f;
    for (int j = 0; j < G; ++j) {
        const size_t uh = (size_t)u * Hq + (size_t)g * G + j;
        const float a = expf(logits[uh * n + key] - lse[uh]);
        acc += (a + epsilon) * sqrtf(fmaxf(wo_norm2[uh * n + key], 0.f));   // rounding can leave -0 or a tiny negative
    }
    if (group_mode == EA_GROUP_MEAN_PROB) acc *= 1.0f / (float)G;
    scores[(size_t)ug * n + key] = acc;
}

// Gram matrix of head j's slice of the output projection: M_j[c, e] = sum_a W_o[a, j*d + c] W_o[a, j*d + e].
// One CTA per (set, head, 16 x 16 block of M_j); done once per model, not on the scoring path.
__global__ void __launch_bounds__(256)
wo_gram_kernel(const __nv_bfloat16* __restrict__ w_o, int d_model, int Hq, int d, float* __restrict__ gram) {
    __shared__ float a_s[16][17], b_s[16][17];
    const int blocks = d / 16;
    const int bc = blockIdx.x / blocks, be = blockIdx.x % blocks;
    const int j = blockIdx.y, set = blockIdx.z;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
    const __nv_bfloat16* W = w_o + (size_t)set * d_model * Hq * d + (size_t)j * d;
    float acc = 0.f;
    for (int a0 = 0; a0 < d_model; a0 += 16) {
        const int a = a0 + ty;
        a_s[ty][tx] = a < d_model ? __bfloat162float(W[(size_t)a * Hq * d + bc * 16 + tx]) : 0.f;
        b_s[ty][tx] = a < d_model ? __bfloat162float(W[(size_t)a * Hq * d + be * 16 + tx]) : 0.f;
        __syncthreads();
#pragma unroll
        for (int r = 0; r < 16; ++r) acc = fmaf(a_s[r][ty], b_s[r][tx], acc);
        __syncthreads();
    }
    gram[(((size_t)set * Hq + j) * d + bc * 16 + ty) * d + be * 16 + tx] = acc;
}

// One thread per softmax row: combine the (max, sum of exp) partials of its work units in order.
__global__ void lse_combine_kernel(const float* __restrict__ lse_part, int n_rows, int n_chunks,
                                   float* __restrict__ lse) {
    const int r = blockIdx.x * blockDim.x + threadIdx.x;
    if (r >= n_rows) return;
    const float* pp = lse_part + (size_t)r * n_chunks * 2;
    float m = -INFINITY, l = 0.f;
    for (int c = 0; c < n_chunks; ++c) {
        const float mo = pp[2 * c], lo = pp[2 * c + 1];
        const float mn = fmaxf(m, mo);
        l = mn == -INFINITY ? 0.f : l * expf(m - mn) + lo * expf(mo - mn);
        m = mn;
    }
    lse[r] = m + logf(l);
}

}  // namespace

ea_status ea_launch_finalize(const ea_ctx* ctx, const ea_shape& s, const float* logits,
                             const __nv_bfloat16* v, float epsilon, float* lse, bool lse_ready, float* scores,
                             cudaStream_t st) {
    const int G = s.n_q_heads / s.n_kv_heads;
    if (lse_ready) {
        // the log-sum-exp of every softmax row was assembled from the log-score kernel's partials
    } else if (s.group_mode == EA_GROUP_MEAN_LOGIT)
        lse_kernel<<<s.n_units * s.n_kv_heads, kLseThreads, 0, st>>>(logits, s.n_keys, G, lse);
    else
        lse_kernel<<<s.n_units * s.n_q_heads, kLseThreads, 0, st>>>(logits, s.n_keys, 1, lse);
    const int keys_per_cta = kFinThreads;   // 8 warps x 32 keys
    dim3 grid((unsigned)((s.n_keys + keys_per_cta - 1) / keys_per_cta),
              (unsigned)(s.n_units * s.n_kv_heads));
    switch (s.head_dim) {
        case 64:
            finalize_kernel<64><<<grid, kFinThreads, 0, st>>>(logits, lse, v, s.n_q_heads, s.n_kv_heads,
                                                             s.n_keys, ea_kv_cap(s), s.group_mode, epsilon, scores);
            break;
        case 128:
            finalize_kernel<128><<<grid, kFinThreads, 0, st>>>(logits, lse, v, s.n_q_heads,
                                                              s.n_kv_heads, s.n_keys, ea_kv_cap(s), s.group_mode,
                                                              epsilon, scores);
            break;
        case 256:
            finalize_kernel<256><<<grid, kFinThreads, 0, st>>>(logits, lse, v, s.n_q_heads,
                                                              s.n_kv_heads, s.n_keys, ea_kv_cap(s), s.group_mode,
                                                              epsilon, scores);
            break;
        default:
            return EA_ERR_UNSUPPORTED;
    }
    ea_count_launches(ctx, lse_ready ? 1 : 2);
    return EA_CHECK_LAUNCH();
}


ea_status ea_launch_vnorm(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* v, int n_ctas, float* vnorm,
                          cudaStream_t st) {
    const long long n_rows = (long long)s.n_units * s.n_kv_heads * s.n_keys;
    const int smem = kVnSmem;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)n_ctas);
    cfg.blockDim = dim3(kVnThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    // clusters of two keep both SMs of a pair for this kernel, so that the CTA pairs of the log-score
    // kernel find whole pairs among the others
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = n_ctas % 2 == 0 ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    cudaError_t err;
    switch (s.head_dim) {
        case 64:
            EA_CUDA_TRY(cudaFuncSetAttribute(vnorm_stream_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            err = cudaLaunchKernelEx(&cfg, vnorm_stream_kernel<64>, v, n_rows, vnorm, ctx->status_dev);
            break;
        case 128:
            EA_CUDA_TRY(cudaFuncSetAttribute(vnorm_stream_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            err = cudaLaunchKernelEx(&cfg, vnorm_stream_kernel<128>, v, n_rows, vnorm, ctx->status_dev);
            break;
        case 256:
            EA_CUDA_TRY(cudaFuncSetAttribute(vnorm_stream_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem));
            err = cudaLaunchKernelEx(&cfg, vnorm_stream_kernel<256>, v, n_rows, vnorm, ctx->status_dev);
            break;
        default:
            return EA_ERR_UNSUPPORTED;
    }
    EA_CUDA_TRY(err);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_weight(const ea_ctx* ctx, const ea_shape& s, const float* logits, const float* lse,
                           const float* vnorm, int vn_stride, float epsilon, float* scores, cudaStream_t st) {
    dim3 grid((unsigned)((s.n_keys + 255) / 256), (unsigned)(s.n_units * s.n_kv_heads));
    weight_kernel<<<grid, 256, 0, st>>>(logits, lse, vnorm, vn_stride, s.n_q_heads, s.n_kv_heads, s.n_keys,
                                        s.group_mode, epsilon, scores);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_vnorm_rows(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* v, int first_row,
                               int n_rows, float* v_norm, cudaStream_t st) {
    const long long total = (long long)s.n_units * s.n_kv_heads * n_rows;
    if (total <= 0) return EA_OK;
    const int lpr = s.head_dim / 8;
    const long long want = (total * lpr + 255) / 256, lim = (long long)ctx->sm_count * 16;
    const unsigned grid = (unsigned)(want < lim ? want : lim);
    const int cap = ea_kv_cap(s);
    switch (s.head_dim) {
        case 64: vnorm_rows_kernel<64><<<grid, 256, 0, st>>>(v, cap, first_row, n_rows, total, v_norm); break;
        case 128: vnorm_rows_kernel<128><<<grid, 256, 0, st>>>(v, cap, first_row, n_rows, total, v_norm); break;
        case 256: vnorm_rows_kernel<256><<<grid, 256, 0, st>>>(v, cap, first_row, n_rows, total, v_norm); break;
        default: return EA_ERR_UNSUPPORTED;
    }
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_lse_combine(const ea_ctx* ctx, const ea_shape& s, const float* lse_part, int n_chunks,
                                float* lse, cudaStream_t st) {
    const int rows = s.n_units * s.n_q_heads;
    lse_combine_kernel<<<(rows + 127) / 128, 128, 0, st>>>(lse_part, rows, n_chunks, lse);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_lse(const ea_ctx* ctx, const ea_shape& s, const float* logits, float* lse, cudaStream_t st) {
    lse_kernel<<<s.n_units * s.n_q_heads, kLseThreads, 0, st>>>(logits, s.n_keys, 1, lse);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_lse_grouped(const ea_ctx* ctx, const ea_shape& s, const float* logits, float* lse, cudaStream_t st) {
    lse_kernel<<<s.n_units * s.n_kv_heads, kLseThreads, 0, st>>>(logits, s.n_keys, s.n_q_heads / s.n_kv_heads, lse);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_finalize_wo(const ea_ctx* ctx, const ea_shape& s, const float* logits, const float* lse,
                                const float* wo_norm2, float epsilon, float* scores, cudaStream_t st) {
    dim3 grid((unsigned)((s.n_keys + 255) / 256), (unsigned)(s.n_units * s.n_kv_heads));
    finalize_wo_kernel<<<grid, 256, 0, st>>>(logits, lse, wo_norm2, s.n_q_heads, s.n_kv_heads, s.n_keys,
                                             s.group_mode, epsilon, scores);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_wo_gram(const ea_ctx* ctx, const __nv_bfloat16* w_o, int d_model, int n_sets, int Hq, int d,
                            float* gram, cudaStream_t st) {
    const int blocks = d / 16;
    dim3 grid((unsigned)(blocks * blocks), (unsigned)Hq, (unsigned)n_sets);
    if (grid.y > 65535u || grid.z > 65535u) return EA_ERR_UNSUPPORTED;
    wo_gram_kernel<<<grid, 256, 0, st>>>(w_o, d_model, Hq, d, gram);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}
