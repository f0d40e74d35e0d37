// ea_compress_host: the whole routine on host buffers, chunk by chunk, with the
// host<->device copies of neighbouring chunks overlapping the kernels.
#include "ea_internal.h"

namespace {

struct staging_plan {
    size_t q, k, v, pos, mu, sigma, scores, idx, k_out, v_out, total;
};

staging_plan plan_staging(const ea_shape& s, int n_kept, int chunk) {
    staging_plan p;
    const size_t C = (size_t)chunk, Hq = (size_t)s.n_q_heads, Hkv = (size_t)s.n_kv_heads;
    const size_t n = (size_t)s.n_keys, d = (size_t)s.head_dim, W = (size_t)s.window;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off = ea_align_up(off + bytes, 256); return at; };
    p.q = take(C * Hq * W * d * 2);
    p.k = take(C * Hkv * n * d * 2);
    p.v = take(C * Hkv * n * d * 2);
    p.pos = take(C * sizeof(int64_t));
    p.mu = take(C * Hq * d * 4);
    p.sigma = take(C * Hq * d * d * 4);
    p.scores = take(C * Hkv * n * 4);
    p.idx = take(C * Hkv * (size_t)n_kept * 4);
    p.k_out = take(C * Hkv * (size_t)n_kept * d * 2);
    p.v_out = take(C * Hkv * (size_t)n_kept * d * 2);
    p.total = off;
    return p;
}

ea_status ensure_host_pipeline(ea_ctx* ctx) {
    if (ctx->host_ready) return EA_OK;
    EA_CUDA_TRY(cudaStreamCreateWithFlags(&ctx->st_h2d, cudaStreamNonBlocking));
    EA_CUDA_TRY(cudaStreamCreateWithFlags(&ctx->st_d2h, cudaStreamNonBlocking));
    EA_CUDA_TRY(cudaEventCreateWithFlags(&ctx->ev_entry, cudaEventDisableTiming));
    for (int b = 0; b < 2; ++b) {
        EA_CUDA_TRY(cudaEventCreateWithFlags(&ctx->ev_h2d[b], cudaEventDisableTiming));
        EA_CUDA_TRY(cudaEventCreateWithFlags(&ctx->ev_comp[b], cudaEventDisableTiming));
        EA_CUDA_TRY(cudaEventCreateWithFlags(&ctx->ev_d2h[b], cudaEventDisableTiming));
    }
    ctx->host_ready = true;
    return EA_OK;
}

}  // namespace

extern "C" {

ea_status ea_host_workspace_bytes(const ea_shape* shape, int32_t n_kept, int32_t units_per_chunk,
                                  size_t* out_bytes) {
    if (!shape || !out_bytes || units_per_chunk < 1) return EA_ERR_INVALID_ARG;
    if (n_kept < 0 || n_kept > shape->n_keys) return EA_ERR_INVALID_ARG;
    ea_shape sub = *shape;
    sub.n_units = units_per_chunk;
    size_t kernel_ws = 0;
    ea_status st = ea_workspace_bytes(&sub, &kernel_ws);
    if (st != EA_OK) return st;
    *out_bytes = ea_align_up(kernel_ws, 256) + 2 * plan_staging(*shape, n_kept, units_per_chunk).total;
    return EA_OK;
}

ea_status ea_compress_host(ea_ctx* ctx, const ea_shape* shape, const void* q_win, const void* k,
                           const void* v, const int64_t* pos_next, int32_t n_future,
                           double rope_base, float epsilon, int32_t n_kept, int32_t units_per_chunk,
                           int32_t* kept_idx, void* k_out, void* v_out, float* scores_opt,
                           void* cuda_stream) {
    if (!ctx || !shape) return EA_ERR_INVALID_ARG;
    size_t need = 0;
    ea_status st = ea_host_workspace_bytes(shape, n_kept, units_per_chunk, &need);
    if (st != EA_OK) return st;
    if (shape->n_units == 0) return EA_OK;
    if (!q_win || !k || !v || !pos_next || !kept_idx || !k_out || !v_out) return EA_ERR_INVALID_ARG;
    if (shape->n_keys < 1 || shape->window < 1 || n_future < 1) return EA_ERR_INVALID_ARG;
    if (shape->kv_capacity != 0 && shape->kv_capacity != shape->n_keys) return EA_ERR_UNSUPPORTED;   // host arrays are dense
    if (ctx->workspace_bytes < need) return EA_ERR_WORKSPACE;

    int prev = 0;
    EA_CUDA_TRY(cudaGetDevice(&prev));
    if (prev != ctx->device) EA_CUDA_TRY(cudaSetDevice(ctx->device));
    st = ensure_host_pipeline(ctx);
    if (st != EA_OK) { if (prev != ctx->device) cudaSetDevice(prev); return st; }

    const staging_plan sp = plan_staging(*shape, n_kept, units_per_chunk);
    ea_shape sub = *shape;
    sub.n_units = units_per_chunk;
    size_t kernel_ws = 0;
    ea_workspace_bytes(&sub, &kernel_ws);
    kernel_ws = ea_align_up(kernel_ws, 256);
    // The device calls use the front of the workspace; staging sits behind it.
    char* base = static_cast<char*>(ctx->workspace) + kernel_ws;
    const size_t saved_ws = ctx->workspace_bytes;

    cudaStream_t main = static_cast<cudaStream_t>(cuda_stream);
    const size_t Hq = (size_t)shape->n_q_heads, Hkv = (size_t)shape->n_kv_heads;
    const size_t n = (size_t)shape->n_keys, d = (size_t)shape->head_dim, W = (size_t)shape->window;
    const size_t q_unit = Hq * W * d * 2, kv_unit = Hkv * n * d * 2;
    const size_t idx_unit = Hkv * (size_t)n_kept * 4, out_unit = Hkv * (size_t)n_kept * d * 2;
    const size_t sc_unit = Hkv * n * 4;

    bool ok = cudaEventRecord(ctx->ev_entry, main) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(ctx->st_h2d, ctx->ev_entry, 0) == cudaSuccess;
    ok = ok && cudaStreamWaitEvent(ctx->st_d2h, ctx->ev_entry, 0) == cudaSuccess;

    int chunk_no = 0;
    for (int u0 = 0; ok && st == EA_OK && u0 < shape->n_units; u0 += units_per_chunk, ++chunk_no) {
        const int b = chunk_no & 1;
        const size_t C = (size_t)((shape->n_units - u0 < units_per_chunk) ? shape->n_units - u0
                                                                          : units_per_chunk);
        char* sb = base + (size_t)b * sp.total;
        // host -> device, once the kernels of the chunk that used this buffer are done
        if (chunk_no >= 2) ok = ok && cudaStreamWaitEvent(ctx->st_h2d, ctx->ev_comp[b], 0) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(sb + sp.q, static_cast<const char*>(q_win) + (size_t)u0 * q_unit,
                                   C * q_unit, cudaMemcpyHostToDevice, ctx->st_h2d) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(sb + sp.k, static_cast<const char*>(k) + (size_t)u0 * kv_unit,
                                   C * kv_unit, cudaMemcpyHostToDevice, ctx->st_h2d) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(sb + sp.v, static_cast<const char*>(v) + (size_t)u0 * kv_unit,
                                   C * kv_unit, cudaMemcpyHostToDevice, ctx->st_h2d) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(sb + sp.pos, pos_next + u0, C * sizeof(int64_t),
                                   cudaMemcpyHostToDevice, ctx->st_h2d) == cudaSuccess;
        ok = ok && cudaEventRecord(ctx->ev_h2d[b], ctx->st_h2d) == cudaSuccess;
        // kernels, once the inputs have landed and this buffer's previous results have left
        ok = ok && cudaStreamWaitEvent(main, ctx->ev_h2d[b], 0) == cudaSuccess;
        if (chunk_no >= 2) ok = ok && cudaStreamWaitEvent(main, ctx->ev_d2h[b], 0) == cudaSuccess;
        if (!ok) break;
        sub.n_units = (int32_t)C;
        ctx->workspace_bytes = kernel_ws;      // the device calls may only use the front part
        st = ea_query_stats(ctx, &sub, sb + sp.q, reinterpret_cast<const int64_t*>(sb + sp.pos), n_future,
                            rope_base, reinterpret_cast<float*>(sb + sp.mu),
                            reinterpret_cast<float*>(sb + sp.sigma), main);
        if (st == EA_OK)
            st = ea_score(ctx, &sub, sb + sp.k, sb + sp.v, reinterpret_cast<float*>(sb + sp.mu),
                          reinterpret_cast<float*>(sb + sp.sigma), epsilon,
                          reinterpret_cast<float*>(sb + sp.scores), nullptr, main);
        if (st == EA_OK)
            st = ea_select_compact(ctx, &sub, reinterpret_cast<float*>(sb + sp.scores), n_kept, sb + sp.k,
                                   sb + sp.v, reinterpret_cast<int32_t*>(sb + sp.idx), sb + sp.k_out,
                                   sb + sp.v_out, main);
        ctx->workspace_bytes = saved_ws;
        if (st != EA_OK) break;
        ok = ok && cudaEventRecord(ctx->ev_comp[b], main) == cudaSuccess;
        // device -> host
        ok = ok && cudaStreamWaitEvent(ctx->st_d2h, ctx->ev_comp[b], 0) == cudaSuccess;
        if (n_kept > 0) {
            ok = ok && cudaMemcpyAsync(reinterpret_cast<char*>(kept_idx) + (size_t)u0 * idx_unit, sb + sp.idx,
                                       C * idx_unit, cudaMemcpyDeviceToHost, ctx->st_d2h) == cudaSuccess;
            ok = ok && cudaMemcpyAsync(static_cast<char*>(k_out) + (size_t)u0 * out_unit, sb + sp.k_out,
                                       C * out_unit, cudaMemcpyDeviceToHost, ctx->st_d2h) == cudaSuccess;
            ok = ok && cudaMemcpyAsync(static_cast<char*>(v_out) + (size_t)u0 * out_unit, sb + sp.v_out,
                                       C * out_unit, cudaMemcpyDeviceToHost, ctx->st_d2h) == cudaSuccess;
        }
        if (scores_opt)
            ok = ok && cudaMemcpyAsync(reinterpret_cast<char*>(scores_opt) + (size_t)u0 * sc_unit,
                                       sb + sp.scores, C * sc_unit, cudaMemcpyDeviceToHost,
                                       ctx->st_d2h) == cudaSuccess;
        ok = ok && cudaEventRecord(ctx->ev_d2h[b], ctx->st_d2h) == cudaSuccess;
    }
    // the caller's stream finishes only after the last results are on the host
    if (ok && st == EA_OK) {
        const int used = chunk_no < 2 ? chunk_no : 2;
        for (int b = 0; b < used; ++b) ok = ok && cudaStreamWaitEvent(main, ctx->ev_d2h[b], 0) == cudaSuccess;
    }
    if (prev != ctx->device) cudaSetDevice(prev);
    if (st != EA_OK) return st;
    return ok ? EA_OK : EA_ERR_CUDA;
}

}  // extern "C"
