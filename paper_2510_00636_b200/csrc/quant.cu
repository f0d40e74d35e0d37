// Quantised cache: keys and values stored as FP8 E4M3 codes with fp32 scales (the paper's Related
// Works call quantisation combinable with eviction; the format is this library's reading):
//     k[u,g,i,c] = decode(k_q8[u,g,i,c]) * k_scale[u,g,c]        one scale per channel
//     v[u,g,i,c] = decode(v_q8[u,g,i,c]) * v_scale[u,g,i]        one scale per token
// Eq. 7 on such keys needs no scaled key at all: mu.k = (s*mu).x and k^T Sigma k = x^T (diag(s) Sigma diag(s)) x
// for the code row x, so the scales are folded into the covariance image and the linear term, and the
// log-score kernel runs on the codes widened to bf16 (every E4M3 value is a bf16 value).  Eq. 9's norm
// is ||v_i|| = v_scale_i ||x_i||, and compaction moves code rows and the value scales of their tokens.
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include "ea_internal.h"

namespace {

// two E4M3 codes -> two floats (exact)
__device__ __forceinline__ float2 e4m3x2_to_float2(uint16_t two) {
    const __half2_raw h = __nv_cvt_fp8x2_to_halfraw2(static_cast<__nv_fp8x2_storage_t>(two), __NV_E4M3);
    return __half22float2(*reinterpret_cast<const __half2*>(&h));
}

// 16 codes per thread -> 16 bf16
__global__ void dequant_k_kernel(const uint4* __restrict__ k_q8, long long pieces, uint4* __restrict__ k_codes) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < pieces; t += stride) {
        const uint4 x = __ldg(k_q8 + t);
        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
        uint32_t o[8];
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            const float2 a = e4m3x2_to_float2((uint16_t)(w[q] & 0xffffu));
            const float2 b = e4m3x2_to_float2((uint16_t)(w[q] >> 16));
            // exact: the float's low 16 bits are zero
            o[2 * q] = (__float_as_uint(a.x) >> 16) | (__float_as_uint(a.y) & 0xffff0000u);
            o[2 * q + 1] = (__float_as_uint(b.x) >> 16) | (__float_as_uint(b.y) & 0xffff0000u);
        }
        k_codes[2 * t] = make_uint4(o[0], o[1], o[2], o[3]);
        k_codes[2 * t + 1] = make_uint4(o[4], o[5], o[6], o[7]);
    }
}

constexpr int kFq8Threads = 256;

// finalize_kernel on value codes: one warp per 32 consecutive keys; a row is D bytes = D / 16 pieces.
template <int D>
__global__ void __launch_bounds__(kFq8Threads)
finalize_q8_kernel(const float* __restrict__ logits, const float* __restrict__ lse, const uint8_t* __restrict__ v_q8,
                   const float* __restrict__ v_scale, int Hq, int Hkv, int n, int cap, int group_mode, float epsilon,
                   float* __restrict__ scores) {
    constexpr int LPR = D / 16;         // lanes per value row (one uint4 = 16 codes each)
    constexpr int RPS = 32 / LPR;       // rows per load step
    constexpr int STEPS = 32 / RPS;
    const int G = Hq / Hkv;
    const int ug = blockIdx.y;
    const int u = ug / Hkv, g = ug % Hkv;
    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const int key0 = (blockIdx.x * (kFq8Threads / 32) + warp) * 32;
    if (key0 >= n) return;
    const uint4* vrow = reinterpret_cast<const uint4*>(v_q8 + ((size_t)ug * cap + key0) * D);      // heads are cap rows apart
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
                const float2 a = e4m3x2_to_float2((uint16_t)(w[q] & 0xffffu));
                const float2 b = e4m3x2_to_float2((uint16_t)(w[q] >> 16));
                ss = fmaf(a.x, a.x, ss);
                ss = fmaf(a.y, a.y, ss);
                ss = fmaf(b.x, b.x, ss);
                ss = fmaf(b.y, b.y, ss);
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
    scores[(size_t)ug * n + key] = (a + epsilon) * (v_scale[(size_t)ug * cap + key] * sqrtf(my_sumsq));
}

// rows of D codes = D / 16 pieces of 16 bytes; the value scale of a token follows its row
__global__ void gather_q8_kernel(const int32_t* __restrict__ kept_idx, long long n_rows_out, int cap, int n_kept, int lpr,
                                 const uint4* __restrict__ k, const uint4* __restrict__ v,
                                 const float* __restrict__ v_scale, uint4* __restrict__ k_out,
                                 uint4* __restrict__ v_out, float* __restrict__ v_scale_out) {
    const long long total = n_rows_out * lpr;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        const long long row = t / lpr;
        const int piece = (int)(t % lpr);
        const long long head = row / n_kept;
        const long long src = head * cap + kept_idx[row];          // heads are cap rows apart in the cache
        k_out[t] = __ldg(k + src * lpr + piece);
        v_out[t] = __ldg(v + src * lpr + piece);
        if (piece == 0) v_scale_out[row] = v_scale[src];
    }
}

// gather_q8_kernel after head-adaptive eviction: output row j of unit u belongs to the head whose range
// [head_off[g], head_off[g + 1]) holds j
__global__ void gather_adaptive_q8_kernel(const int32_t* __restrict__ kept_idx, const int32_t* __restrict__ head_off,
                                          long long n_rows_out, int cap, int Hkv, int unit_stride, int lpr,
                                          const uint4* __restrict__ k, const uint4* __restrict__ v,
                                          const float* __restrict__ v_scale, uint4* __restrict__ k_out,
                                          uint4* __restrict__ v_out, float* __restrict__ v_scale_out) {
    const long long total = n_rows_out * lpr;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        const long long row = t / lpr;
        const int piece = (int)(t % lpr);
        const long long u = row / unit_stride;
        const int j = (int)(row % unit_stride);
        const int32_t* off = head_off + u * (Hkv + 1);
        int lo = 0, hi = Hkv - 1;                      // the last g with off[g] <= j
        while (lo < hi) {
            const int mid = (lo + hi + 1) / 2;
            if (off[mid] <= j) lo = mid;
            else hi = mid - 1;
        }
        const long long src = (u * Hkv + lo) * cap + kept_idx[row];
        k_out[t] = __ldg(k + src * lpr + piece);
        v_out[t] = __ldg(v + src * lpr + piece);
        if (piece == 0) v_scale_out[row] = v_scale[src];
    }
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

ea_status ea_launch_dequant_k(const ea_ctx* ctx, const ea_shape& s, const uint8_t* k_q8, __nv_bfloat16* k_codes,
                              cudaStream_t st) {
    // every row of the buffers, so that the scratch has the cache's own strides
    const long long pieces = (long long)s.n_units * s.n_kv_heads * ea_kv_cap(s) * (s.head_dim / 16);
    long long want = (pieces + 255) / 256;
    const long long cap = (long long)ctx->sm_count * 16;
    dequant_k_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(reinterpret_cast<const uint4*>(k_q8), pieces,
                                                                          reinterpret_cast<uint4*>(k_codes));
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_finalize_q8(const ea_ctx* ctx, const ea_shape& s, const float* logits, const float* lse,
                                const uint8_t* v_q8, const float* v_scale, float epsilon, float* scores,
                                cudaStream_t st) {
    dim3 grid((unsigned)((s.n_keys + kFq8Threads - 1) / kFq8Threads), (unsigned)(s.n_units * s.n_kv_heads));
    switch (s.head_dim) {
        case 64:
            finalize_q8_kernel<64><<<grid, kFq8Threads, 0, st>>>(logits, lse, v_q8, v_scale, s.n_q_heads, s.n_kv_heads,
                                                                 s.n_keys, ea_kv_cap(s), s.group_mode, epsilon, scores);
            break;
        case 128:
            finalize_q8_kernel<128><<<grid, kFq8Threads, 0, st>>>(logits, lse, v_q8, v_scale, s.n_q_heads, s.n_kv_heads,
                                                                  s.n_keys, ea_kv_cap(s), s.group_mode, epsilon, scores);
            break;
        case 256:
            finalize_q8_kernel<256><<<grid, kFq8Threads, 0, st>>>(logits, lse, v_q8, v_scale, s.n_q_heads, s.n_kv_heads,
                                                                  s.n_keys, ea_kv_cap(s), s.group_mode, epsilon, scores);
            break;
        default:
            return EA_ERR_UNSUPPORTED;
    }
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_gather_q8(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* kept_idx,
                              const uint8_t* k_q8, const uint8_t* v_q8, const float* v_scale, uint8_t* k_out,
                              uint8_t* v_out, float* v_scale_out, cudaStream_t st) {
    if (n_kept <= 0) return EA_OK;
    const int lpr = s.head_dim / 16;
    const long long rows = (long long)s.n_units * s.n_kv_heads * n_kept;
    long long want = (rows * lpr + 255) / 256;
    const long long cap = (long long)ctx->sm_count * 16;
    gather_q8_kernel<<<(unsigned)(want < cap ? want : cap), 256, 0, st>>>(
        kept_idx, rows, ea_kv_cap(s), n_kept, lpr, reinterpret_cast<const uint4*>(k_q8), reinterpret_cast<const uint4*>(v_q8),
        v_scale, reinterpret_cast<uint4*>(k_out), reinterpret_cast<uint4*>(v_out), v_scale_out);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

extern "C" {

ea_status ea_score_q8_scratch_bytes(const ea_shape* shape, size_t* bytes) {
    if (!shape || !bytes) return EA_ERR_INVALID_ARG;
    size_t need = 0;
    const ea_status st = ea_workspace_bytes(shape, &need);    // validates the shape
    if (st != EA_OK) return st;
    *bytes = ea_mma_q8_supported(*shape)
                 ? 0
                 : (size_t)shape->n_units * shape->n_kv_heads * ea_kv_cap(*shape) * shape->head_dim * sizeof(__nv_bfloat16);
    return EA_OK;
}

ea_status ea_score_q8(ea_ctx* ctx, const ea_shape* shape, const void* k_q8, const float* k_scale, const void* v_q8,
                      const float* v_scale, const float* mu_bar, const float* sigma_bar, float epsilon,
                      void* k_scratch, float* scores, float* logits_opt, void* cuda_stream) {
    if (!ctx || !shape) return EA_ERR_INVALID_ARG;
    size_t need = 0;
    ea_status st = ea_workspace_bytes(shape, &need);          // validates the shape
    if (st != EA_OK) return st;
    if (shape->n_units == 0 || shape->n_keys == 0) return EA_OK;
    if (!k_q8 || !k_scale || !v_q8 || !v_scale || !mu_bar || !sigma_bar || !scores) return EA_ERR_INVALID_ARG;
    if (!k_scratch && !ea_mma_q8_supported(*shape)) return EA_ERR_INVALID_ARG;
    if (!aligned16(k_q8) || !aligned16(v_q8) || !aligned16(k_scratch) || !aligned16(mu_bar) || !aligned16(sigma_bar) ||
        !aligned16(scores) || !aligned16(logits_opt))
        return EA_ERR_INVALID_ARG;
    if (!(epsilon >= 0.0f)) return EA_ERR_INVALID_ARG;
    if (ctx->workspace_bytes < need) return EA_ERR_WORKSPACE;
    const ea_ws_plan plan = ea_plan_workspace(*shape);
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    char* ws = static_cast<char*>(ctx->workspace);
    float* logits = logits_opt ? logits_opt : reinterpret_cast<float*>(ws + plan.logits);
    float* lse = reinterpret_cast<float*>(ws + plan.lse);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    __nv_bfloat16* codes = static_cast<__nv_bfloat16*>(k_scratch);
    ea_quad_form eq7 = ea_eq7_form(*shape, mu_bar, sigma_bar);
    ctx->image_ready = false;                         // this call writes its own (scaled) images into the workspace
    eq7.ch_scale = k_scale;
    bool lse_ready = false;
    if (ea_mma_q8_supported(*shape)) {
        // the tensor-core kernel takes the codes as they are and widens them itself
        float* lse_part = reinterpret_cast<float*>(ws + plan.lse_part);
        int n_chunks = 0;
        st = ea_launch_logits_mma_q8(ctx, *shape, static_cast<const uint8_t*>(k_q8), eq7, ws + plan.image,
                                     reinterpret_cast<float*>(ws + plan.vec), logits, lse_part, &n_chunks, stream);
        if (st == EA_OK && shape->group_mode != EA_GROUP_MEAN_LOGIT) {
            st = ea_launch_lse_combine(ctx, *shape, lse_part, n_chunks, lse, stream);
            lse_ready = true;
        }
    } else {
        // otherwise a pass of its own widens the codes into the caller's scratch first
        st = ea_launch_dequant_k(ctx, *shape, static_cast<const uint8_t*>(k_q8), codes, stream);
    }
    if (st == EA_OK && !ea_mma_q8_supported(*shape)) {
        if (ea_mma_path_supported(*shape)) {
            float* lse_part = reinterpret_cast<float*>(ws + plan.lse_part);
            int n_chunks = 0;
            st = ea_launch_logits_mma(ctx, *shape, codes, eq7, ws + plan.image, reinterpret_cast<float*>(ws + plan.vec),
                                      logits, lse_part, &n_chunks, stream);
            if (st == EA_OK && shape->group_mode != EA_GROUP_MEAN_LOGIT) {
                st = ea_launch_lse_combine(ctx, *shape, lse_part, n_chunks, lse, stream);
                lse_ready = true;
            }
        } else {
            st = ea_launch_logits_simt(ctx, *shape, codes, eq7, logits, stream);
        }
    }
    if (st == EA_OK && !lse_ready) {
        // one softmax row per query head, or per KV head for the mean of the log-scores
        if (shape->group_mode == EA_GROUP_MEAN_LOGIT) st = ea_launch_lse_grouped(ctx, *shape, logits, lse, stream);
        else st = ea_launch_lse(ctx, *shape, logits, lse, stream);
    }
    if (st == EA_OK)
        st = ea_launch_finalize_q8(ctx, *shape, logits, lse, static_cast<const uint8_t*>(v_q8), v_scale, epsilon, scores,
                                   stream);
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_select_compact_q8(ea_ctx* ctx, const ea_shape* shape, const float* scores, int32_t n_kept,
                               const void* k_q8, const void* v_q8, const float* v_scale, int32_t* kept_idx,
                               void* k_out, void* v_out, float* v_scale_out, void* cuda_stream) {
    if (!ctx || !shape) return EA_ERR_INVALID_ARG;
    size_t need = 0;
    ea_status st = ea_workspace_bytes(shape, &need);
    if (st != EA_OK) return st;
    if (n_kept < 0 || n_kept > shape->n_keys) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_kept == 0) return EA_OK;
    if (!scores || !kept_idx || !k_q8 || !v_q8 || !v_scale || !k_out || !v_out || !v_scale_out) return EA_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(k_q8) || !aligned16(v_q8) || !aligned16(k_out) || !aligned16(v_out))
        return EA_ERR_INVALID_ARG;
    {
        const size_t in_bytes = (size_t)shape->n_units * shape->n_kv_heads * ea_kv_cap(*shape) * shape->head_dim;
        const size_t out_bytes = (size_t)shape->n_units * shape->n_kv_heads * n_kept * shape->head_dim;
        const char* ins[2] = {static_cast<const char*>(k_q8), static_cast<const char*>(v_q8)};
        const char* outs[2] = {static_cast<const char*>(k_out), static_cast<const char*>(v_out)};
        for (const char* o : outs)
            for (const char* i : ins)
                if (o < i + in_bytes && i < o + out_bytes) return EA_ERR_INVALID_ARG;
    }
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = ea_launch_select(ctx, *shape, scores, n_kept, kept_idx, stream);
    if (st == EA_OK)
        st = ea_launch_gather_q8(ctx, *shape, n_kept, kept_idx, static_cast<const uint8_t*>(k_q8),
                                 static_cast<const uint8_t*>(v_q8), v_scale, static_cast<uint8_t*>(k_out),
                                 static_cast<uint8_t*>(v_out), v_scale_out, stream);
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_select_compact_adaptive_q8(ea_ctx* ctx, const ea_shape* shape, const float* scores, int32_t n_kept,
                                        int32_t n_floor, const void* k_q8, const void* v_q8, const float* v_scale,
                                        int32_t* kept_idx, int32_t* head_offsets, void* k_out, void* v_out,
                                        float* v_scale_out, void* cuda_stream) {
    if (!ctx || !shape) return EA_ERR_INVALID_ARG;
    size_t need = 0;
    ea_status st = ea_workspace_bytes(shape, &need);
    if (st != EA_OK) return st;
    if (n_kept < 0 || n_kept > shape->n_keys || n_floor < 0 || n_floor > n_kept) return EA_ERR_INVALID_ARG;
    if ((long long)shape->n_kv_heads * n_kept > 0x7fffffffLL) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0) return EA_OK;
    if (!head_offsets) return EA_ERR_INVALID_ARG;
    if (n_kept > 0 && (!scores || !kept_idx || !k_q8 || !v_q8 || !v_scale || !k_out || !v_out || !v_scale_out))
        return EA_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(k_q8) || !aligned16(v_q8) || !aligned16(k_out) || !aligned16(v_out))
        return EA_ERR_INVALID_ARG;
    if (n_kept > 0) {
        const size_t in_bytes = (size_t)shape->n_units * shape->n_kv_heads * ea_kv_cap(*shape) * shape->head_dim;
        const size_t out_bytes = (size_t)shape->n_units * shape->n_kv_heads * n_kept * shape->head_dim;
        const char* ins[2] = {static_cast<const char*>(k_q8), static_cast<const char*>(v_q8)};
        const char* outs[2] = {static_cast<const char*>(k_out), static_cast<const char*>(v_out)};
        for (const char* o : outs)
            for (const char* i : ins)
                if (o < i + in_bytes && i < o + out_bytes) return EA_ERR_INVALID_ARG;
    }
    if (ctx->workspace_bytes < need) return EA_ERR_WORKSPACE;
    const ea_ws_plan plan = ea_plan_workspace(*shape);
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = ea_launch_select_adaptive(ctx, *shape, scores, n_kept, n_floor,
                                   static_cast<char*>(ctx->workspace) + plan.adaptive, kept_idx, head_offsets, stream);
    if (st == EA_OK && n_kept > 0) {
        const int lpr = shape->head_dim / 16, unit_stride = shape->n_kv_heads * n_kept;
        const long long rows = (long long)shape->n_units * unit_stride;
        const long long want = (rows * lpr + 255) / 256, lim = (long long)ctx->sm_count * 16;
        gather_adaptive_q8_kernel<<<(unsigned)(want < lim ? want : lim), 256, 0, stream>>>(
            kept_idx, head_offsets, rows, ea_kv_cap(*shape), shape->n_kv_heads, unit_stride, lpr,
            static_cast<const uint4*>(k_q8), static_cast<const uint4*>(v_q8), v_scale, static_cast<uint4*>(k_out),
            static_cast<uint4*>(v_out), v_scale_out);
        ea_count_launches(ctx, 1);
        st = EA_CHECK_LAUNCH();
    }
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_select_compact_inplace_q8(ea_ctx* ctx, const ea_shape* shape, const float* scores, int32_t n_kept,
                                       void* k_q8, void* v_q8, float* v_scale, int32_t* kept_idx, int32_t unordered,
                                       void* cuda_stream) {
    if (!ctx || !shape) return EA_ERR_INVALID_ARG;
    size_t need = 0;
    ea_status st = ea_workspace_bytes(shape, &need);
    if (st != EA_OK) return st;
    if (n_kept < 0 || n_kept > shape->n_keys) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_kept == 0) return EA_OK;
    if (!scores || !kept_idx || !k_q8 || !v_q8 || !v_scale) return EA_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(k_q8) || !aligned16(v_q8)) return EA_ERR_INVALID_ARG;
    if (unordered && 2 * (size_t)n_kept * sizeof(int32_t) > 200 * 1024) return EA_ERR_UNSUPPORTED;
    {
        const size_t bytes = (size_t)shape->n_units * shape->n_kv_heads * ea_kv_cap(*shape) * shape->head_dim;
        const char* a = static_cast<const char*>(k_q8);
        const char* b = static_cast<const char*>(v_q8);
        if (a < b + bytes && b < a + bytes) return EA_ERR_INVALID_ARG;      // K and V are distinct buffers
    }
    if (unordered && ctx->workspace_bytes < need) return EA_ERR_WORKSPACE;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (unordered) {
        // the ascending selection goes to the workspace (the log-score region: nothing of a compaction reads it)
        const ea_ws_plan plan = ea_plan_workspace(*shape);
        int32_t* sel = reinterpret_cast<int32_t*>(static_cast<char*>(ctx->workspace) + plan.logits);
        st = ea_launch_select(ctx, *shape, scores, n_kept, sel, stream);
        if (st == EA_OK) st = ea_launch_compact_fill(ctx, *shape, n_kept, sel, kept_idx, k_q8, v_q8, stream, true);
        // the value scales follow their rows (kept_idx now names the original row at each position)
        if (st == EA_OK) st = ea_launch_carry_f32(ctx, *shape, n_kept, kept_idx, v_scale, stream);
    } else {
        st = ea_launch_select(ctx, *shape, scores, n_kept, kept_idx, stream);
        if (st == EA_OK) st = ea_launch_compact_inplace(ctx, *shape, n_kept, kept_idx, k_q8, v_q8, stream, true);
        if (st == EA_OK) st = ea_launch_carry_f32(ctx, *shape, n_kept, kept_idx, v_scale, stream);
    }
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

}  // extern "C"
