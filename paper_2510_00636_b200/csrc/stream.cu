// Streaming decode (the decoding set-up of Sec. 4: a buffer of the most recent hidden states or
// queries, compression every few hundred generated tokens down to a fixed budget): the pieces that
// let ONE cache buffer and ONE window buffer live through consecutive compression events.
//
//   ea_cache_append      new K/V rows go behind the n_keys rows a head holds in its fixed range
//   ea_window_push       new pre-RoPE queries go into a ring of `window` rows per query head
//   ea_query_stats_ring  Eq. 5 / Eq. 6 over whatever the ring holds (partly filled or wrapped)
// Everything is stream work on device-resident state (the ring's fill counter lives in device
// memory), so a whole event - append, push, statistics, ea_score, ea_select_compact_inplace - can be
// captured once per shape and replayed.
#include "ea_internal.h"

namespace {

// rows_new[u, g, j, :] -> cache[(u * Hkv + g) * cap + n_old + j, :], 16 bytes per thread
__global__ void cache_append_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new, long long pieces,
                                    int n_new, int n_old, int cap, int lpr, uint4* __restrict__ k, uint4* __restrict__ v) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < pieces; t += stride) {
        const long long row = t / lpr;
        const int piece = (int)(t % lpr);
        const long long head = row / n_new;
        const int j = (int)(row % n_new);
        const long long dst = ((head * cap + n_old + j) * lpr) + piece;
        k[dst] = __ldg(k_new + t);
        v[dst] = __ldg(v_new + t);
    }
}

// q_new[u, h, j, :] -> ring[(u * Hq + h) * W + (pushed[u] + j) % W, :]; when more than W rows arrive at once only
// the last W are written (the earlier ones would be overwritten anyway)
__global__ void window_push_kernel(const uint4* __restrict__ q_new, long long pieces, int n_new, int Hq, int W, int lpr,
                                   const long long* __restrict__ pushed, uint4* __restrict__ ring) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    const int skip = n_new > W ? n_new - W : 0;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < pieces; t += stride) {
        const long long row = t / lpr;
        const int piece = (int)(t % lpr);
        const long long uh = row / n_new;
        const int j = (int)(row % n_new);
        if (j < skip) continue;
        const long long at = (pushed[uh / Hq] + j) % W;
        ring[(uh * W + at) * lpr + piece] = __ldg(q_new + t);
    }
}

// the value scales of appended code rows: scale_new[head, j] -> scale[head * cap + n_old + j]
__global__ void scale_append_kernel(const float* __restrict__ scale_new, long long total, int n_new, int n_old, int cap,
                                    float* __restrict__ scale) {
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride)
        scale[(t / n_new) * cap + n_old + t % n_new] = scale_new[t];
}

__global__ void window_bump_kernel(long long* __restrict__ pushed, int n_units, int n_new) {
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u < n_units) pushed[u] += n_new;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

ea_status check_common(const ea_ctx* ctx, const ea_shape* s) {
    if (!ctx || !s) return EA_ERR_INVALID_ARG;
    if (s->n_units < 0 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->n_keys < 0 || s->window < 0)
        return EA_ERR_INVALID_ARG;
    if (s->n_q_heads % s->n_kv_heads != 0) return EA_ERR_INVALID_ARG;
    if (s->head_dim != 64 && s->head_dim != 128 && s->head_dim != 256) return EA_ERR_UNSUPPORTED;
    if ((long long)s->n_units * s->n_q_heads > 65535LL) return EA_ERR_UNSUPPORTED;
    return EA_OK;
}

unsigned grid_for(const ea_ctx* ctx, long long pieces) {
    const long long want = (pieces + 255) / 256, cap = (long long)ctx->sm_count * 16;
    return (unsigned)(want < cap ? (want > 0 ? want : 1) : cap);
}

}  // namespace

extern "C" {

ea_status ea_cache_append(ea_ctx* ctx, const ea_shape* shape, void* k, void* v, const void* k_new, const void* v_new,
                          int32_t n_new, void* cuda_stream) {
    ea_status st = check_common(ctx, shape);
    if (st != EA_OK) return st;
    const int cap = ea_kv_cap(*shape);
    if (n_new < 0 || (long long)shape->n_keys + n_new > cap) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_new == 0) return EA_OK;
    if (!k || !v || !k_new || !v_new) return EA_ERR_INVALID_ARG;
    if (!aligned16(k) || !aligned16(v) || !aligned16(k_new) || !aligned16(v_new)) return EA_ERR_INVALID_ARG;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    const int lpr = shape->head_dim / 8;
    const long long pieces = (long long)shape->n_units * shape->n_kv_heads * n_new * lpr;
    cache_append_kernel<<<grid_for(ctx, pieces), 256, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), pieces, n_new, shape->n_keys, cap, lpr,
        static_cast<uint4*>(k), static_cast<uint4*>(v));
    ea_count_launches(ctx, 1);
    st = EA_CHECK_LAUNCH();
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_cache_append_q8(ea_ctx* ctx, const ea_shape* shape, void* k_q8, void* v_q8, float* v_scale,
                             const void* k_new, const void* v_new, const float* v_scale_new, int32_t n_new,
                             void* cuda_stream) {
    ea_status st = check_common(ctx, shape);
    if (st != EA_OK) return st;
    const int cap = ea_kv_cap(*shape);
    if (n_new < 0 || (long long)shape->n_keys + n_new > cap) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_new == 0) return EA_OK;
    if (!k_q8 || !v_q8 || !v_scale || !k_new || !v_new || !v_scale_new) return EA_ERR_INVALID_ARG;
    if (!aligned16(k_q8) || !aligned16(v_q8) || !aligned16(k_new) || !aligned16(v_new)) return EA_ERR_INVALID_ARG;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int lpr = shape->head_dim / 16;                       // a row of codes is head_dim bytes
    const long long rows = (long long)shape->n_units * shape->n_kv_heads * n_new, pieces = rows * lpr;
    cache_append_kernel<<<grid_for(ctx, pieces), 256, 0, stream>>>(
        static_cast<const uint4*>(k_new), static_cast<const uint4*>(v_new), pieces, n_new, shape->n_keys, cap, lpr,
        static_cast<uint4*>(k_q8), static_cast<uint4*>(v_q8));
    scale_append_kernel<<<grid_for(ctx, rows), 256, 0, stream>>>(v_scale_new, rows, n_new, shape->n_keys, cap, v_scale);
    ea_count_launches(ctx, 2);
    st = EA_CHECK_LAUNCH();
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_window_push(ea_ctx* ctx, const ea_shape* shape, void* q_ring, int64_t* ring_pushed, const void* q_new,
                         int32_t n_new, void* cuda_stream) {
    ea_status st = check_common(ctx, shape);
    if (st != EA_OK) return st;
    if (n_new < 0 || shape->window < 1) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_new == 0) return EA_OK;
    if (!q_ring || !ring_pushed || !q_new) return EA_ERR_INVALID_ARG;
    if (!aligned16(q_ring) || !aligned16(q_new)) return EA_ERR_INVALID_ARG;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int lpr = shape->head_dim / 8;
    const long long pieces = (long long)shape->n_units * shape->n_q_heads * n_new * lpr;
    window_push_kernel<<<grid_for(ctx, pieces), 256, 0, stream>>>(
        static_cast<const uint4*>(q_new), pieces, n_new, shape->n_q_heads, shape->window, lpr,
        reinterpret_cast<const long long*>(ring_pushed), static_cast<uint4*>(q_ring));
    // the counters move only after every row has been placed relative to their old values
    window_bump_kernel<<<(shape->n_units + 127) / 128, 128, 0, stream>>>(reinterpret_cast<long long*>(ring_pushed),
                                                                        shape->n_units, n_new);
    ea_count_launches(ctx, 2);
    st = EA_CHECK_LAUNCH();
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_query_stats_ring(ea_ctx* ctx, const ea_shape* shape, const void* q_ring, const int64_t* ring_pushed,
                              const int64_t* pos_next, int32_t n_future, double rope_base, float* mu_bar,
                              float* sigma_bar, void* cuda_stream) {
    ea_status st = check_common(ctx, shape);
    if (st != EA_OK) return st;
    if (shape->rope_layout != EA_ROPE_HALF_SPLIT && shape->rope_layout != EA_ROPE_INTERLEAVED)
        return EA_ERR_INVALID_ARG;
    if (shape->cov_norm != EA_COV_POPULATION && shape->cov_norm != EA_COV_SAMPLE) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0) return EA_OK;
    if (!q_ring || !ring_pushed || !pos_next || !mu_bar) return EA_ERR_INVALID_ARG;
    if (!aligned16(q_ring) || !aligned16(mu_bar) || !aligned16(sigma_bar)) return EA_ERR_INVALID_ARG;
    if (n_future < 1 || !(rope_base > 0.0) || shape->window < 1) return EA_ERR_INVALID_ARG;
    const ea_ws_plan plan = ea_plan_workspace(*shape);
    if (ctx->workspace_bytes < plan.logits /* rope_coef region only */) return EA_ERR_WORKSPACE;
    void* image = nullptr;
    float* vec = nullptr;
    if (!ea_fused_image_target(ctx, *shape, &image, &vec)) return EA_ERR_WORKSPACE;
    if (!sigma_bar && !image) return EA_ERR_INVALID_ARG;       // sigma_bar may only be left out in fused mode
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    float* coef = reinterpret_cast<float*>(static_cast<char*>(ctx->workspace) + plan.rope_coef);
    st = ea_launch_stats_ring(ctx, *shape, static_cast<const __nv_bfloat16*>(q_ring), ring_pushed, pos_next, n_future,
                              rope_base, coef, mu_bar, sigma_bar, static_cast<cudaStream_t>(cuda_stream), image, vec);
    if (st != EA_OK) ctx->image_ready = false;
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

}  // extern "C"
