// Host side of the C ABI: argument validation, workspace planning, context
// lifetime, and the order of kernel launches of each call.
#include <stdio.h>
#include <string.h>

#include <new>

#include "ea_internal.h"

namespace {

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

ea_status check_shape(const ea_shape* s) {
    if (!s) return EA_ERR_INVALID_ARG;
    if (s->n_units < 0 || s->n_q_heads < 1 || s->n_kv_heads < 1 || s->n_keys < 0 || s->window < 0)
        return EA_ERR_INVALID_ARG;
    if (s->n_q_heads % s->n_kv_heads != 0) return EA_ERR_INVALID_ARG;
    if (s->rope_layout != EA_ROPE_HALF_SPLIT && s->rope_layout != EA_ROPE_INTERLEAVED)
        return EA_ERR_INVALID_ARG;
    if (s->group_mode < EA_GROUP_MEAN_PROB || s->group_mode > EA_GROUP_MEAN_LOGIT)
        return EA_ERR_INVALID_ARG;
    if (s->cov_norm != EA_COV_POPULATION && s->cov_norm != EA_COV_SAMPLE) return EA_ERR_INVALID_ARG;
    if (s->kv_capacity != 0 && s->kv_capacity < s->n_keys) return EA_ERR_INVALID_ARG;
    if (s->head_dim != 64 && s->head_dim != 128 && s->head_dim != 256) return EA_ERR_UNSUPPORTED;
    // several kernels put one (unit, head) per gridDim.y entry
    if ((long long)s->n_units * s->n_q_heads > 65535LL) return EA_ERR_UNSUPPORTED;
    return EA_OK;
}

thread_local char g_last_cuda_error[192] = "";

}  // namespace

// Fused statistics: where the images of `s` go, or nullptr when this call does not write them.
bool ea_fused_image_target(ea_ctx* ctx, const ea_shape& s, void** image, float** vec) {
    *image = nullptr;
    *vec = nullptr;
    ctx->image_ready = false;                          // whatever the workspace held is stale after a statistics call
    if (!ctx->fused_stats) return true;
    if (s.head_dim > 128 || !ea_mma_path_supported(s) || s.group_mode == EA_GROUP_MEAN_LOGIT) return true;
    const ea_ws_plan plan = ea_plan_workspace(s);
    if (ctx->workspace_bytes < plan.total) return false;
    *image = static_cast<char*>(ctx->workspace) + plan.image;
    *vec = reinterpret_cast<float*>(static_cast<char*>(ctx->workspace) + plan.vec);
    ctx->image_ready = true;
    ctx->image_shape = s;
    return true;
}

void ea_note_cuda_error(cudaError_t err, const char* file, int line) {
    const char* base = file;
    for (const char* c = file; *c; ++c)
        if (*c == '/') base = c + 1;
    snprintf(g_last_cuda_error, sizeof(g_last_cuda_error), "%s (%s) at %s:%d", cudaGetErrorName(err),
             cudaGetErrorString(err), base, line);
}

ea_ws_plan ea_plan_workspace(const ea_shape& s) {
    ea_ws_plan p;
    size_t off = 0;
    const size_t U = (size_t)s.n_units, Hq = (size_t)s.n_q_heads;
    const size_t n = (size_t)s.n_keys, d = (size_t)s.head_dim;
    p.rope_coef = off;  off = ea_align_up(off + U * (d / 2) * 2 * sizeof(float), 256);
    p.logits = off;     off = ea_align_up(off + U * Hq * n * sizeof(float), 256);
    p.lse = off;        off = ea_align_up(off + U * Hq * sizeof(float), 256);
    const bool mma = ea_mma_path_supported(s);
    p.image = off;      off = ea_align_up(off + (mma ? ea_mma_image_bytes(s) : 0), 1024);
    p.vec = off;        off = ea_align_up(off + (mma ? ea_mma_vec_bytes(s) : 0), 256);
    p.lse_part = off;   off = ea_align_up(off + (mma ? ea_mma_lse_part_bytes(s) : 0), 256);
    p.vnorm = off;      off = ea_align_up(off + (mma ? U * (size_t)s.n_kv_heads * n * sizeof(float) : 0), 256);
    p.adaptive = off;   off = ea_align_up(off + ea_adaptive_ws_bytes(s), 256);
    p.total = off;
    return p;
}

extern "C" {

const char* ea_version(void) { return "ea-b200 0.2"; }

const char* ea_last_cuda_error(void) { return g_last_cuda_error; }

const char* ea_status_string(ea_status s) {
    switch (s) {
        case EA_OK: return "EA_OK";
        case EA_ERR_INVALID_ARG: return "EA_ERR_INVALID_ARG";
        case EA_ERR_UNSUPPORTED: return "EA_ERR_UNSUPPORTED";
        case EA_ERR_WORKSPACE: return "EA_ERR_WORKSPACE";
        case EA_ERR_CUDA: return "EA_ERR_CUDA";
        case EA_ERR_NOT_SM100: return "EA_ERR_NOT_SM100";
        case EA_ERR_DEVICE_TIMEOUT: return "EA_ERR_DEVICE_TIMEOUT";
    }
    return "EA_ERR_UNKNOWN";
}

ea_status ea_workspace_bytes(const ea_shape* shape, size_t* out_bytes) {
    if (!out_bytes) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    *out_bytes = ea_plan_workspace(*shape).total;
    return EA_OK;
}

int64_t ea_n_kept(int64_t n_keys, double compression_ratio) {
    if (n_keys <= 0) return 0;
    const double x = (double)n_keys * (1.0 - compression_ratio);
    if (!(x > 0.0)) return 0;
    if (x >= (double)n_keys) return n_keys;
    return (int64_t)x;
}

ea_status ea_create(ea_ctx** out_ctx, int device, size_t workspace_bytes) {
    if (!out_ctx) return EA_ERR_INVALID_ARG;
    *out_ctx = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess) { cudaGetLastError(); return EA_ERR_CUDA; }
    if (device < 0 || device >= count) return EA_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    EA_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10) return EA_ERR_NOT_SM100;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    EA_CUDA_TRY(cudaSetDevice(device));
    ea_ctx* ctx = new (std::nothrow) ea_ctx();
    if (!ctx) { cudaSetDevice(prev); return EA_ERR_CUDA; }
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->sm_budget = ctx->sm_count;
    ctx->side_sms = 0;
    ctx->side_ready = false;
    ctx->fused_stats = false;
    ctx->image_ready = false;
    ctx->workspace = nullptr;
    ctx->workspace_bytes = workspace_bytes;
    ctx->status_host = nullptr;
    ctx->status_dev = nullptr;
    ctx->host_ready = false;
    ctx->profiling = false;
    ctx->launches = 0;
    ctx->n_events = 0;
    ctx->n_events_created = 0;
    ctx->ev_start = new (std::nothrow) cudaEvent_t[kMaxProfileEvents];
    ctx->ev_stop = new (std::nothrow) cudaEvent_t[kMaxProfileEvents];
    bool ok = ctx->ev_start && ctx->ev_stop;
    if (ok && workspace_bytes > 0) ok = cudaMalloc(&ctx->workspace, workspace_bytes) == cudaSuccess;
    if (ok) ok = cudaHostAlloc((void**)&ctx->status_host, sizeof(int), cudaHostAllocMapped) == cudaSuccess;
    if (ok) {
        *ctx->status_host = 0;
        ok = cudaHostGetDevicePointer((void**)&ctx->status_dev, ctx->status_host, 0) == cudaSuccess;
    }
    if (!ok) {
        cudaGetLastError();
        if (ctx->workspace) cudaFree(ctx->workspace);
        if (ctx->status_host) cudaFreeHost(ctx->status_host);
        delete[] ctx->ev_start;
        delete[] ctx->ev_stop;
        delete ctx;
        cudaSetDevice(prev);
        return EA_ERR_CUDA;
    }
    cudaSetDevice(prev);
    *out_ctx = ctx;
    return EA_OK;
}

ea_status ea_destroy(ea_ctx* ctx) {
    if (!ctx) return EA_OK;
    int prev = 0;
    cudaGetDevice(&prev);
    cudaSetDevice(ctx->device);
    if (ctx->workspace) cudaFree(ctx->workspace);
    if (ctx->status_host) cudaFreeHost(ctx->status_host);
    if (ctx->side_ready) {
        cudaStreamDestroy(ctx->st_side);
        cudaEventDestroy(ctx->ev_fork);
        cudaEventDestroy(ctx->ev_join);
    }
    if (ctx->host_ready) {
        cudaStreamDestroy(ctx->st_h2d);
        cudaStreamDestroy(ctx->st_d2h);
        cudaEventDestroy(ctx->ev_entry);
        for (int b = 0; b < 2; ++b) {
            cudaEventDestroy(ctx->ev_h2d[b]);
            cudaEventDestroy(ctx->ev_comp[b]);
            cudaEventDestroy(ctx->ev_d2h[b]);
        }
    }
    for (int i = 0; i < ctx->n_events_created; ++i) {
        cudaEventDestroy(ctx->ev_start[i]);
        cudaEventDestroy(ctx->ev_stop[i]);
    }
    delete[] ctx->ev_start;
    delete[] ctx->ev_stop;
    cudaSetDevice(prev);
    delete ctx;
    return EA_OK;
}

ea_status ea_query_stats(ea_ctx* ctx, const ea_shape* shape, const void* q_win,
                         const int64_t* pos_next, int32_t n_future, double rope_base,
                         float* mu_bar, float* sigma_bar, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (shape->n_units == 0) return EA_OK;
    if (!q_win || !pos_next || !mu_bar) return EA_ERR_INVALID_ARG;
    if (!aligned16(q_win) || !aligned16(mu_bar) || !aligned16(sigma_bar)) return EA_ERR_INVALID_ARG;
    if (n_future < 1 || !(rope_base > 0.0)) return EA_ERR_INVALID_ARG;
    if (shape->window < 1 || (shape->cov_norm == EA_COV_SAMPLE && shape->window < 2))
        return EA_ERR_INVALID_ARG;
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
    st = ea_launch_stats(ctx, *shape, static_cast<const __nv_bfloat16*>(q_win), pos_next, n_future,
                         rope_base, coef, mu_bar, sigma_bar, static_cast<cudaStream_t>(cuda_stream), image, vec);
    if (st != EA_OK) ctx->image_ready = false;
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_query_stats_hidden(ea_ctx* ctx, const ea_shape* shape, const void* hidden, const void* w_q,
                                int32_t d_model, int32_t n_weight_sets, float* q_scratch,
                                const int64_t* pos_next, int32_t n_future, double rope_base, float* mu_bar,
                                float* sigma_bar, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (shape->n_units == 0) return EA_OK;
    if (!hidden || !w_q || !q_scratch || !pos_next || !mu_bar || !sigma_bar) return EA_ERR_INVALID_ARG;
    if (!aligned16(hidden) || !aligned16(w_q) || !aligned16(q_scratch) || !aligned16(mu_bar) ||
        !aligned16(sigma_bar))
        return EA_ERR_INVALID_ARG;
    if (n_future < 1 || !(rope_base > 0.0)) return EA_ERR_INVALID_ARG;
    if (shape->window < 1 || (shape->cov_norm == EA_COV_SAMPLE && shape->window < 2))
        return EA_ERR_INVALID_ARG;
    if (d_model < 8 || d_model % 8 != 0) return EA_ERR_INVALID_ARG;
    if (n_weight_sets < 1 || shape->n_units % n_weight_sets != 0) return EA_ERR_INVALID_ARG;
    if (!ea_project_supported(*shape, d_model)) return EA_ERR_UNSUPPORTED;
    const ea_ws_plan plan = ea_plan_workspace(*shape);
    if (ctx->workspace_bytes < plan.logits /* rope_coef region only */) return EA_ERR_WORKSPACE;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    float* coef = reinterpret_cast<float*>(static_cast<char*>(ctx->workspace) + plan.rope_coef);
    st = ea_launch_project(ctx, *shape, static_cast<const __nv_bfloat16*>(hidden),
                           static_cast<const __nv_bfloat16*>(w_q), d_model, n_weight_sets, q_scratch, stream);
    if (st == EA_OK)
        st = ea_launch_stats_f32(ctx, *shape, q_scratch, pos_next, n_future, rope_base, coef, mu_bar, sigma_bar,
                                 stream);
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

// ea_score and ea_score_vnorm: exactly one of v (the value rows) and v_norm (their norms, carried with the
// cache, [units, Hkv, capacity]) is given.
static ea_status score_impl(ea_ctx* ctx, const ea_shape* shape, const void* k, const void* v, const float* v_norm,
                            const float* mu_bar, const float* sigma_bar, float epsilon, float* scores,
                            float* logits_opt, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (shape->n_units == 0 || shape->n_keys == 0) return EA_OK;
    if (!k || (!v && !v_norm) || !scores) return EA_ERR_INVALID_ARG;
    // sigma_bar == NULL: the images the last statistics call of this context wrote for this very shape
    // (ea_set_fused_stats) stand in for mu_bar and sigma_bar
    const bool from_image = sigma_bar == nullptr;
    if (from_image) {
        ea_shape a = *shape, b = ctx->image_shape;
        a.window = b.window = 0;                                // the window length does not shape the images
        if (!ctx->image_ready || memcmp(&a, &b, sizeof(ea_shape)) != 0) return EA_ERR_INVALID_ARG;
    } else if (!mu_bar) {
        return EA_ERR_INVALID_ARG;
    }
    if (!aligned16(k) || !aligned16(v) || !aligned16(mu_bar) || !aligned16(sigma_bar) ||
        !aligned16(scores) || !aligned16(logits_opt))
        return EA_ERR_INVALID_ARG;
    if (!(epsilon >= 0.0f)) return EA_ERR_INVALID_ARG;
    const ea_ws_plan plan = ea_plan_workspace(*shape);
    if (ctx->workspace_bytes < plan.total) return EA_ERR_WORKSPACE;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    char* ws = static_cast<char*>(ctx->workspace);
    float* logits = logits_opt ? logits_opt : reinterpret_cast<float*>(ws + plan.logits);
    float* lse = reinterpret_cast<float*>(ws + plan.lse);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
    const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(v);
    const ea_quad_form eq7 = ea_eq7_form(*shape, from_image ? nullptr : mu_bar, sigma_bar);
    if (!from_image) ctx->image_ready = false;       // the images are rebuilt from the statistics given here
    if (ea_mma_path_supported(*shape) && shape->group_mode != EA_GROUP_MEAN_LOGIT) {
        // tensor-core log-scores with the log-sum-exp partials from their epilogue
        float* lse_part = reinterpret_cast<float*>(ws + plan.lse_part);
        float* vnorm = reinterpret_cast<float*>(ws + plan.vnorm);
        int n_chunks = 0;
        const bool side = v && ctx->side_sms > 0 && ea_kv_cap(*shape) == shape->n_keys;   // the side pass streams a dense V
        if (side) {
            // the value norms do not depend on the log-scores: their pass over V goes to a few SMs of its
            // own, on a second stream, and is launched first so that it is resident when the log-score
            // kernel takes the others
            EA_CUDA_TRY(cudaEventRecord(ctx->ev_fork, stream));
            EA_CUDA_TRY(cudaStreamWaitEvent(ctx->st_side, ctx->ev_fork, 0));
            st = ea_launch_vnorm(ctx, *shape, vb, ctx->side_sms, vnorm, ctx->st_side);
            if (st == EA_OK) EA_CUDA_TRY(cudaEventRecord(ctx->ev_join, ctx->st_side));
        }
        if (st == EA_OK)
            st = ea_launch_logits_mma(ctx, *shape, kb, eq7, ws + plan.image,
                                      reinterpret_cast<float*>(ws + plan.vec), logits, lse_part, &n_chunks, stream);
        if (st == EA_OK) st = ea_launch_lse_combine(ctx, *shape, lse_part, n_chunks, lse, stream);
        if (side) {
            // always rejoin, whatever happened in between: the caller's stream must not run ahead of the side pass
            EA_CUDA_TRY(cudaStreamWaitEvent(stream, ctx->ev_join, 0));
            if (st == EA_OK) st = ea_launch_weight(ctx, *shape, logits, lse, vnorm, shape->n_keys, epsilon, scores, stream);
        } else if (st == EA_OK && v_norm) {
            st = ea_launch_weight(ctx, *shape, logits, lse, v_norm, ea_kv_cap(*shape), epsilon, scores, stream);
        } else if (st == EA_OK) {
            st = ea_launch_finalize(ctx, *shape, logits, vb, epsilon, lse, true, scores, stream);
        }
    } else {
        if (ea_mma_path_supported(*shape)) {
            int n_chunks = 0;
            st = ea_launch_logits_mma(ctx, *shape, kb, eq7, ws + plan.image,
                                      reinterpret_cast<float*>(ws + plan.vec), logits,
                                      reinterpret_cast<float*>(ws + plan.lse_part), &n_chunks, stream);
        } else {
            st = ea_launch_logits_simt(ctx, *shape, kb, eq7, logits, stream);
        }
        if (st == EA_OK && v_norm) {
            // one softmax row per query head, or per KV head for the mean of the log-scores
            st = shape->group_mode == EA_GROUP_MEAN_LOGIT ? ea_launch_lse_grouped(ctx, *shape, logits, lse, stream)
                                                          : ea_launch_lse(ctx, *shape, logits, lse, stream);
            if (st == EA_OK)
                st = ea_launch_weight(ctx, *shape, logits, lse, v_norm, ea_kv_cap(*shape), epsilon, scores, stream);
        } else if (st == EA_OK) {
            st = ea_launch_finalize(ctx, *shape, logits, vb, epsilon, lse, false, scores, stream);
        }
    }
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_score(ea_ctx* ctx, const ea_shape* shape, const void* k, const void* v,
                   const float* mu_bar, const float* sigma_bar, float epsilon, float* scores,
                   float* logits_opt, void* cuda_stream) {
    return score_impl(ctx, shape, k, v, nullptr, mu_bar, sigma_bar, epsilon, scores, logits_opt, cuda_stream);
}

ea_status ea_score_vnorm(ea_ctx* ctx, const ea_shape* shape, const void* k, const float* v_norm,
                         const float* mu_bar, const float* sigma_bar, float epsilon, float* scores,
                         float* logits_opt, void* cuda_stream) {
    return score_impl(ctx, shape, k, nullptr, v_norm, mu_bar, sigma_bar, epsilon, scores, logits_opt, cuda_stream);
}

ea_status ea_value_norms(ea_ctx* ctx, const ea_shape* shape, const void* v, int32_t first_row, int32_t n_rows,
                         float* v_norm, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (first_row < 0 || n_rows < 0 || (long long)first_row + n_rows > ea_kv_cap(*shape)) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_rows == 0) return EA_OK;
    if (!v || !v_norm || !aligned16(v)) return EA_ERR_INVALID_ARG;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    st = ea_launch_vnorm_rows(ctx, *shape, static_cast<const __nv_bfloat16*>(v), first_row, n_rows, v_norm,
                              static_cast<cudaStream_t>(cuda_stream));
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_carry_f32_inplace(ea_ctx* ctx, const ea_shape* shape, const int32_t* kept_idx, int32_t n_kept,
                               float* values, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (n_kept < 0 || n_kept > shape->n_keys) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_kept == 0) return EA_OK;
    if (!kept_idx || !values) return EA_ERR_INVALID_ARG;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    st = ea_launch_carry_f32(ctx, *shape, n_kept, kept_idx, values, static_cast<cudaStream_t>(cuda_stream));
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_wo_gram(ea_ctx* ctx, const void* w_o, int32_t d_model, int32_t n_weight_sets, int32_t n_q_heads,
                     int32_t head_dim, float* wo_gram, void* cuda_stream) {
    if (!ctx || !w_o || !wo_gram) return EA_ERR_INVALID_ARG;
    if (d_model < 1 || n_weight_sets < 1 || n_q_heads < 1) return EA_ERR_INVALID_ARG;
    if (head_dim != 64 && head_dim != 128 && head_dim != 256) return EA_ERR_INVALID_ARG;
    if (!aligned16(w_o) || !aligned16(wo_gram)) return EA_ERR_INVALID_ARG;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    const ea_status st = ea_launch_wo_gram(ctx, static_cast<const __nv_bfloat16*>(w_o), d_model, n_weight_sets,
                                           n_q_heads, head_dim, wo_gram, static_cast<cudaStream_t>(cuda_stream));
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_score_wo(ea_ctx* ctx, const ea_shape* shape, const void* k, const void* v, const float* mu_bar,
                      const float* sigma_bar, const float* wo_gram, int32_t n_weight_sets, float epsilon,
                      float* wo_scratch, float* scores, float* logits_opt, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (shape->group_mode == EA_GROUP_MEAN_LOGIT) return EA_ERR_UNSUPPORTED;   // the weighting is per query head
    if (shape->n_units == 0 || shape->n_keys == 0) return EA_OK;
    if (!k || !v || !mu_bar || !sigma_bar || !wo_gram || !wo_scratch || !scores) return EA_ERR_INVALID_ARG;
    if (!aligned16(k) || !aligned16(v) || !aligned16(mu_bar) || !aligned16(sigma_bar) || !aligned16(wo_gram) ||
        !aligned16(wo_scratch) || !aligned16(scores) || !aligned16(logits_opt))
        return EA_ERR_INVALID_ARG;
    if (!(epsilon >= 0.0f)) return EA_ERR_INVALID_ARG;
    if (n_weight_sets < 1 || shape->n_units % n_weight_sets != 0) return EA_ERR_INVALID_ARG;
    const ea_ws_plan plan = ea_plan_workspace(*shape);
    if (ctx->workspace_bytes < plan.total) return EA_ERR_WORKSPACE;
    ctx->image_ready = false;                         // this call writes its own images into the workspace
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    char* ws = static_cast<char*>(ctx->workspace);
    float* logits = logits_opt ? logits_opt : reinterpret_cast<float*>(ws + plan.logits);
    float* lse = reinterpret_cast<float*>(ws + plan.lse);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const __nv_bfloat16* kb = static_cast<const __nv_bfloat16*>(k);
    const __nv_bfloat16* vb = static_cast<const __nv_bfloat16*>(v);
    const ea_quad_form eq7 = ea_eq7_form(*shape, mu_bar, sigma_bar);
    // ||W_o^h v||^2 = v^T (W_o^h^T W_o^h) v: the same kernels, the value rows in place of the keys
    const ea_quad_form norm2 = {nullptr, wo_gram, shape->n_units / n_weight_sets, 0.0f, 1.0f, nullptr};
    if (ea_mma_path_supported(*shape)) {
        float* lse_part = reinterpret_cast<float*>(ws + plan.lse_part);
        float* vec = reinterpret_cast<float*>(ws + plan.vec);
        int n_chunks = 0;
        st = ea_launch_logits_mma(ctx, *shape, vb, norm2, ws + plan.image, vec, wo_scratch, lse_part, &n_chunks,
                                  stream);
        if (st == EA_OK)
            st = ea_launch_logits_mma(ctx, *shape, kb, eq7, ws + plan.image, vec, logits, lse_part, &n_chunks, stream);
        if (st == EA_OK) st = ea_launch_lse_combine(ctx, *shape, lse_part, n_chunks, lse, stream);
    } else {
        st = ea_launch_logits_simt(ctx, *shape, vb, norm2, wo_scratch, stream);
        if (st == EA_OK) st = ea_launch_logits_simt(ctx, *shape, kb, eq7, logits, stream);
        if (st == EA_OK) st = ea_launch_lse(ctx, *shape, logits, lse, stream);
    }
    if (st == EA_OK) st = ea_launch_finalize_wo(ctx, *shape, logits, lse, wo_scratch, epsilon, scores, stream);
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_select_compact(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                            int32_t n_kept, const void* k, const void* v, int32_t* kept_idx,
                            void* k_out, void* v_out, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (n_kept < 0 || n_kept > shape->n_keys) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_kept == 0) return EA_OK;
    if (!scores || !kept_idx) return EA_ERR_INVALID_ARG;
    const bool do_gather = k_out != nullptr || v_out != nullptr;
    if (do_gather && (!k || !v || !k_out || !v_out)) return EA_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
        return EA_ERR_INVALID_ARG;
    if (do_gather) {
        const size_t in_bytes = (size_t)shape->n_units * shape->n_kv_heads * ea_kv_cap(*shape) *
                                shape->head_dim * sizeof(__nv_bfloat16);
        const size_t out_bytes = (size_t)shape->n_units * shape->n_kv_heads * n_kept *
                                 shape->head_dim * sizeof(__nv_bfloat16);
        const char* ins[2] = {static_cast<const char*>(k), static_cast<const char*>(v)};
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
    if (st == EA_OK && do_gather)
        st = ea_launch_gather(ctx, *shape, n_kept, kept_idx, static_cast<const __nv_bfloat16*>(k),
                              static_cast<const __nv_bfloat16*>(v), static_cast<__nv_bfloat16*>(k_out),
                              static_cast<__nv_bfloat16*>(v_out), stream);
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_select_compact_inplace(ea_ctx* ctx, const ea_shape* shape, const float* scores, int32_t n_kept,
                                    void* k, void* v, int32_t* kept_idx, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (n_kept < 0 || n_kept > shape->n_keys) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_kept == 0) return EA_OK;
    if (!scores || !kept_idx || !k || !v) return EA_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(k) || !aligned16(v)) return EA_ERR_INVALID_ARG;
    {
        const size_t bytes = (size_t)shape->n_units * shape->n_kv_heads * ea_kv_cap(*shape) * shape->head_dim *
                             sizeof(__nv_bfloat16);
        const char* a = static_cast<const char*>(k);
        const char* b = static_cast<const char*>(v);
        if (a < b + bytes && b < a + bytes) return EA_ERR_INVALID_ARG;      // K and V are distinct buffers
    }
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = ea_launch_select(ctx, *shape, scores, n_kept, kept_idx, stream);
    if (st == EA_OK)
        st = ea_launch_compact_inplace(ctx, *shape, n_kept, kept_idx, k, v, stream);
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_select_compact_inplace_unordered(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                                              int32_t n_kept, void* k, void* v, int32_t* kept_idx,
                                              void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (n_kept < 0 || n_kept > shape->n_keys) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0 || n_kept == 0) return EA_OK;
    if (!scores || !kept_idx || !k || !v) return EA_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(k) || !aligned16(v)) return EA_ERR_INVALID_ARG;
    if (2 * (size_t)n_kept * sizeof(int32_t) > 200 * 1024) return EA_ERR_UNSUPPORTED;
    {
        const size_t bytes = (size_t)shape->n_units * shape->n_kv_heads * ea_kv_cap(*shape) * shape->head_dim *
                             sizeof(__nv_bfloat16);
        const char* a = static_cast<const char*>(k);
        const char* b = static_cast<const char*>(v);
        if (a < b + bytes && b < a + bytes) return EA_ERR_INVALID_ARG;      // K and V are distinct buffers
    }
    const ea_ws_plan plan = ea_plan_workspace(*shape);
    if (ctx->workspace_bytes < plan.total) return EA_ERR_WORKSPACE;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // the ascending selection goes to the workspace (the log-score region: nothing of a compaction reads it)
    int32_t* sel = reinterpret_cast<int32_t*>(static_cast<char*>(ctx->workspace) + plan.logits);
    st = ea_launch_select(ctx, *shape, scores, n_kept, sel, stream);
    if (st == EA_OK)
        st = ea_launch_compact_fill(ctx, *shape, n_kept, sel, kept_idx, k, v, stream);
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

ea_status ea_select_compact_adaptive(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                                     int32_t n_kept, int32_t n_floor, const void* k, const void* v,
                                     int32_t* kept_idx, int32_t* head_offsets, void* k_out, void* v_out,
                                     void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ea_status st = check_shape(shape);
    if (st != EA_OK) return st;
    if (n_kept < 0 || n_kept > shape->n_keys || n_floor < 0 || n_floor > n_kept) return EA_ERR_INVALID_ARG;
    if ((long long)shape->n_kv_heads * n_kept > 0x7fffffffLL) return EA_ERR_INVALID_ARG;
    if (shape->n_units == 0) return EA_OK;
    if (!head_offsets) return EA_ERR_INVALID_ARG;
    if (n_kept > 0 && (!scores || !kept_idx)) return EA_ERR_INVALID_ARG;
    const bool do_gather = n_kept > 0 && (k_out != nullptr || v_out != nullptr);
    if (do_gather && (!k || !v || !k_out || !v_out)) return EA_ERR_INVALID_ARG;
    if (!aligned16(scores) || !aligned16(k) || !aligned16(v) || !aligned16(k_out) || !aligned16(v_out))
        return EA_ERR_INVALID_ARG;
    if (do_gather) {
        const size_t in_bytes = (size_t)shape->n_units * shape->n_kv_heads * ea_kv_cap(*shape) *
                                shape->head_dim * sizeof(__nv_bfloat16);
        const size_t out_bytes = (size_t)shape->n_units * shape->n_kv_heads * n_kept *
                                 shape->head_dim * sizeof(__nv_bfloat16);
        const char* ins[2] = {static_cast<const char*>(k), static_cast<const char*>(v)};
        const char* outs[2] = {static_cast<const char*>(k_out), static_cast<const char*>(v_out)};
        for (const char* o : outs)
            for (const char* i : ins)
                if (o < i + in_bytes && i < o + out_bytes) return EA_ERR_INVALID_ARG;
    }
    const ea_ws_plan plan = ea_plan_workspace(*shape);
    if (ctx->workspace_bytes < plan.total) return EA_ERR_WORKSPACE;
    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    st = ea_launch_select_adaptive(ctx, *shape, scores, n_kept, n_floor,
                                   static_cast<char*>(ctx->workspace) + plan.adaptive, kept_idx, head_offsets, stream);
    if (st == EA_OK && do_gather)
        st = ea_launch_gather_adaptive(ctx, *shape, n_kept, kept_idx, head_offsets,
                                       static_cast<const __nv_bfloat16*>(k), static_cast<const __nv_bfloat16*>(v),
                                       static_cast<__nv_bfloat16*>(k_out), static_cast<__nv_bfloat16*>(v_out), stream);
    if (prev != ctx->device) cudaSetDevice(prev);
    return st;
}

int64_t ea_n_floor(int64_t n_kept, double safeguard) {
    const double x = (double)n_kept * safeguard;
    int64_t f = (int64_t)x;
    if (f < 0) f = 0;
    if (f > n_kept) f = n_kept;
    return f;
}

ea_status ea_set_sm_budget(ea_ctx* ctx, int32_t n_sms) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    if (n_sms == 0) n_sms = ctx->sm_count;
    if (n_sms < 32 || n_sms > ctx->sm_count) return EA_ERR_INVALID_ARG;
    ctx->sm_budget = n_sms;
    return EA_OK;
}

ea_status ea_set_fused_stats(ea_ctx* ctx, int32_t on) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ctx->fused_stats = on != 0;
    ctx->image_ready = false;
    return EA_OK;
}

ea_status ea_set_side_sms(ea_ctx* ctx, int32_t n_sms) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    if (n_sms < 0 || n_sms % 2 != 0 || n_sms > ctx->sm_count - 32) return EA_ERR_INVALID_ARG;
    if (n_sms > 0 && !ctx->side_ready) {
        int prev = 0;
        EA_CUDA_TRY(cudaGetDevice(&prev));
        if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
        cudaError_t e = cudaStreamCreateWithFlags(&ctx->st_side, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_join, cudaEventDisableTiming);
        if (prev != ctx->device) cudaSetDevice(prev);
        EA_CUDA_TRY(e);
        ctx->side_ready = true;
    }
    ctx->side_sms = n_sms;
    return EA_OK;
}

ea_status ea_sync_status(ea_ctx* ctx, void* cuda_stream) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    EA_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
    const int s = *ctx->status_host;
    *ctx->status_host = 0;
    return s == 0 ? EA_OK : static_cast<ea_status>(s);
}

ea_status ea_profile_begin(ea_ctx* ctx) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ctx->profiling = true;
    ctx->launches = 0;
    ctx->n_events = 0;
    return EA_OK;
}

ea_status ea_profile_end(ea_ctx* ctx, void* cuda_stream, double* score_kernel_ms,
                         int64_t* timed_launches, int64_t* total_kernel_launches) {
    if (!ctx) return EA_ERR_INVALID_ARG;
    ctx->profiling = false;
    EA_CUDA_TRY(cudaStreamSynchronize(static_cast<cudaStream_t>(cuda_stream)));
    double total = 0.0;
    for (int i = 0; i < ctx->n_events; ++i) {
        float ms = 0.f;
        EA_CUDA_TRY(cudaEventElapsedTime(&ms, ctx->ev_start[i], ctx->ev_stop[i]));
        total += (double)ms;
    }
    if (score_kernel_ms) *score_kernel_ms = total;
    if (timed_launches) *timed_launches = ctx->n_events;
    if (total_kernel_launches) *total_kernel_launches = ctx->launches;
    return EA_OK;
}

}  // extern "C"

cudaEvent_t ea_profile_mark_start(const ea_ctx* cctx, cudaStream_t st) {
    ea_ctx* ctx = const_cast<ea_ctx*>(cctx);
    if (!ctx->profiling || ctx->n_events >= kMaxProfileEvents) return nullptr;
    const int i = ctx->n_events;
    if (i >= ctx->n_events_created) {
        if (cudaEventCreate(&ctx->ev_start[i]) != cudaSuccess) return nullptr;
        if (cudaEventCreate(&ctx->ev_stop[i]) != cudaSuccess) { cudaEventDestroy(ctx->ev_start[i]); return nullptr; }
        ctx->n_events_created = i + 1;
    }
    cudaEventRecord(ctx->ev_start[i], st);
    ctx->n_events = i + 1;
    return ctx->ev_stop[i];
}

void ea_profile_mark_stop(const ea_ctx* ctx, cudaEvent_t stop, cudaStream_t st) {
    (void)ctx;
    if (stop) cudaEventRecord(stop, st);
}
