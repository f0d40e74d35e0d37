// Internal declarations shared by the translation units of libea.so.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <math.h>
#include <stddef.h>
#include <stdint.h>

#include "ea.h"

struct ea_ctx {
    int device;
    int sm_count;        // SMs of the device
    int sm_budget;       // SMs the persistent kernels of this context may occupy (ea_set_sm_budget)
    bool fused_stats;    // ea_set_fused_stats: the statistics calls also write the covariance images
    bool image_ready;    // the workspace holds the images of `image_shape`, written by the last statistics call
    ea_shape image_shape;
    int side_sms;        // SMs of the value-norm pass that runs beside the log-score kernel (0: no side pass)
    bool side_ready;     // side stream and events exist
    cudaStream_t st_side;
    cudaEvent_t ev_fork, ev_join;
    void* workspace;
    size_t workspace_bytes;
    int* status_host;    // pinned, mapped: device kernels write EA_ERR_DEVICE_TIMEOUT here
    int* status_dev;     // device alias of status_host
    // benchmark instrumentation (ea_profile_begin / ea_profile_end)
    bool profiling;
    long long launches;          // kernels launched since ea_profile_begin
    int n_events;                // event pairs recorded in this window
    int n_events_created;        // event pairs that exist
    cudaEvent_t* ev_start;       // [kMaxProfileEvents]
    cudaEvent_t* ev_stop;
    // host-buffer pipeline (ea_compress_host), created on first use
    bool host_ready;
    cudaStream_t st_h2d, st_d2h;
    cudaEvent_t ev_entry, ev_h2d[2], ev_comp[2], ev_d2h[2];
};

constexpr int kMaxProfileEvents = 4096;

// Count `n` kernel launches made on behalf of `ctx`.
static inline void ea_count_launches(const ea_ctx* ctx, int n) {
    const_cast<ea_ctx*>(ctx)->launches += n;
}
// Bracket the dominant kernel with events while profiling; returns the stop event or nullptr.
cudaEvent_t ea_profile_mark_start(const ea_ctx* ctx, cudaStream_t st);
void ea_profile_mark_stop(const ea_ctx* ctx, cudaEvent_t stop, cudaStream_t st);

// Byte offsets of the workspace regions.  Regions of different calls overlap
// on purpose except where one call's output feeds the next.
struct ea_ws_plan {
    size_t rope_coef;    // fp32 [U, d/2, 2]             (ea_query_stats)
    size_t logits;       // fp32 [U, Hq, n]              (ea_score, when logits_opt == NULL)
    size_t lse;          // fp32 [U, Hq]                 (ea_score)
    size_t image;        // bf16 covariance images of the tensor-core log-score kernel (ea_score)
    size_t vec;          // fp32 [U*Hq, d] epilogue vectors of that kernel               (ea_score)
    size_t lse_part;     // fp32 [U*Hq, chunks, 2] log-sum-exp partials of that kernel    (ea_score)
    size_t vnorm;        // fp32 [U, Hkv, n] value norms (ea_score with a side pass, ea_set_side_sms)
    size_t adaptive;     // radix histograms, search state and per-head counts (ea_select_compact_adaptive)
    size_t total;
};

ea_ws_plan ea_plan_workspace(const ea_shape& s);

// The CUDA error behind the calling thread's most recent EA_ERR_CUDA (ea_last_cuda_error).
void ea_note_cuda_error(cudaError_t err, const char* file, int line);
// EA_OK if no runtime call of this thread has failed since the last check, else EA_ERR_CUDA (noted).
static inline ea_status ea_check_launch(const char* file, int line) {
    const cudaError_t err = cudaGetLastError();
    if (err == cudaSuccess) return EA_OK;
    ea_note_cuda_error(err, file, line);
    return EA_ERR_CUDA;
}
#define EA_CHECK_LAUNCH() ea_check_launch(__FILE__, __LINE__)

#define EA_CUDA_TRY(expr)                                   \
    do {                                                    \
        cudaError_t err__ = (expr);                         \
        if (err__ != cudaSuccess) {                         \
            ea_note_cuda_error(err__, __FILE__, __LINE__);  \
            cudaGetLastError();                             \
            return EA_ERR_CUDA;                             \
        }                                                   \
    } while (0)

static inline size_t ea_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
// Rows per KV head in the K/V buffers (the cache is the first n_keys of them).
static inline int ea_kv_cap(const ea_shape& s) { return s.kv_capacity > 0 ? s.kv_capacity : s.n_keys; }

// ---- launchers (each returns EA_OK or EA_ERR_CUDA from cudaGetLastError) ----
// image / vec != nullptr (head_dim <= 128 only): also write the log-score kernel's covariance images; sigma_bar
// may then be nullptr.
ea_status ea_launch_stats(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* q_win,
                          const int64_t* pos_next, int n_future, double rope_base, float* rope_coef,
                          float* mu_bar, float* sigma_bar, cudaStream_t st, void* image = nullptr,
                          float* vec = nullptr);

// The same statistics over a ring of window rows: pushed[u] rows written so far, at most s.window of them valid.
ea_status ea_launch_stats_ring(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* q_ring,
                               const int64_t* pushed, const int64_t* pos_next, int n_future, double rope_base,
                               float* rope_coef, float* mu_bar, float* sigma_bar, cudaStream_t st,
                               void* image = nullptr, float* vec = nullptr);

// Fused statistics (ea_set_fused_stats): the workspace addresses the images of `s` go to, or nullptr when this
// statistics call does not write them; false if the workspace is too small for them.
bool ea_fused_image_target(ea_ctx* ctx, const ea_shape& s, void** image, float** vec);

// What the log-score kernels evaluate per (query head h, row x of the KV head it reads):
//   lin_scale * lin_h . x + quad_scale * x^T quad_h x
// Eq. 7: rows = keys, lin = mu_bar, quad = sigma_bar, scales 1/sqrt(d) and 1/(2d), one matrix per unit;
// ||W_o^h v||^2: rows = values, no linear term, quad = W_o^h^T W_o^h shared by the units of a weight set.
struct ea_quad_form {
    const float* lin;        // fp32 [sets * Hq, d] or nullptr
    const float* quad;       // fp32 [sets * Hq, d, d]
    int units_per_set;       // unit u reads set u / units_per_set
    float lin_scale, quad_scale;
    // rows given as codes x with the real row diag(ch_scale) x (quantised keys): fp32 [units * Hkv, d] or
    // nullptr.  The scales are folded into lin and quad as they are read (lin_c s_c, quad_ac s_a s_c).
    const float* ch_scale;
};
static inline ea_quad_form ea_eq7_form(const ea_shape& s, const float* mu_bar, const float* sigma_bar) {
    ea_quad_form f = {mu_bar, sigma_bar, 1, 1.0f / sqrtf((float)s.head_dim), 0.5f / (float)s.head_dim, nullptr};
    return f;
}

ea_status ea_launch_logits_simt(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* k,
                                const ea_quad_form& form, float* logits, cudaStream_t st);

// bf16 rank-3 TMA tensor map, box (box0 x box1 x 1), 128-byte swizzle, zero fill outside.
bool ea_tensor_map_bf16_3d(CUtensorMap* map, const void* base, uint64_t n0, uint64_t n1, uint64_t n2,
                           uint64_t stride1, uint64_t stride2, uint32_t box0, uint32_t box1, bool bytes_plain = false);

// Window queries from hidden states, Q[u,h,w,:] = W_Q^h H[u,w,:] in fp32 (tcgen05 GEMM).
bool ea_project_supported(const ea_shape& s, int d_model);
ea_status ea_launch_project(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* hidden,
                            const __nv_bfloat16* w_q, int d_model, int n_sets, float* q_win, cudaStream_t st);
// The statistics kernels on fp32 window queries.
ea_status ea_launch_stats_f32(const ea_ctx* ctx, const ea_shape& s, const float* q_win, const int64_t* pos_next,
                              int n_future, double rope_base, float* rope_coef, float* mu_bar, float* sigma_bar,
                              cudaStream_t st);

// Tensor-core log-score kernel (tcgen05): available for some shapes only.
bool ea_mma_path_supported(const ea_shape& s);
size_t ea_mma_image_bytes(const ea_shape& s);
size_t ea_mma_vec_bytes(const ea_shape& s);
size_t ea_mma_lse_part_bytes(const ea_shape& s);
// form.quad == nullptr: the images in `image` / `vec` are already there (fused statistics)
ea_status ea_launch_logits_mma(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* k,
                               const ea_quad_form& form, void* image, float* vec,
                               float* logits, float* lse_part, int* n_chunks, cudaStream_t st);
// The same kernel on FP8 E4M3 key codes, widened to bf16 inside it (head_dim <= 128); form.ch_scale carries the scales.
bool ea_mma_q8_supported(const ea_shape& s);
ea_status ea_launch_logits_mma_q8(const ea_ctx* ctx, const ea_shape& s, const uint8_t* k_q8,
                                  const ea_quad_form& form, void* image, float* vec, float* logits,
                                  float* lse_part, int* n_chunks, cudaStream_t st);
// log-sum-exp per softmax row from the per-work-unit partials of the tensor-core kernel
ea_status ea_launch_lse_combine(const ea_ctx* ctx, const ea_shape& s, const float* lse_part, int n_chunks,
                                float* lse, cudaStream_t st);

// ||v|| of every value row on n_ctas SMs (bulk-copy-fed stream), and the weighting that uses them.
ea_status ea_launch_vnorm(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* v, int n_ctas, float* vnorm,
                          cudaStream_t st);
// (vn_stride: floats between the norms of consecutive heads)
ea_status ea_launch_weight(const ea_ctx* ctx, const ea_shape& s, const float* logits, const float* lse,
                           const float* vnorm, int vn_stride, float epsilon, float* scores, cudaStream_t st);
// ||v|| of rows first_row .. first_row + n_rows - 1 of every head, into v_norm [units, Hkv, capacity]
ea_status ea_launch_vnorm_rows(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* v, int first_row,
                               int n_rows, float* v_norm, cudaStream_t st);
// values[head][j] <- values[head][idx[head][j]] for j < n_kept (idx[j] >= j), values [units, Hkv, capacity]
ea_status ea_launch_carry_f32(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* idx, float* values,
                              cudaStream_t st);

ea_status ea_launch_finalize(const ea_ctx* ctx, const ea_shape& s, const float* logits,
                             const __nv_bfloat16* v, float epsilon, float* lse, bool lse_ready, float* scores,
                             cudaStream_t st);

// Eq. 9 with the output projection: Gram matrices of the per-head slices of W_o, and the
// weighting (1/G) sum_h (a_hat_h + eps) sqrt(wo_norm2_h).
ea_status ea_launch_wo_gram(const ea_ctx* ctx, const __nv_bfloat16* w_o, int d_model, int n_sets, int Hq, int d,
                            float* gram, cudaStream_t st);
ea_status ea_launch_lse(const ea_ctx* ctx, const ea_shape& s, const float* logits, float* lse, cudaStream_t st);
// one softmax row per KV head over the mean of its group's log-scores (EA_GROUP_MEAN_LOGIT)
ea_status ea_launch_lse_grouped(const ea_ctx* ctx, const ea_shape& s, const float* logits, float* lse, cudaStream_t st);
ea_status ea_launch_finalize_wo(const ea_ctx* ctx, const ea_shape& s, const float* logits, const float* lse,
                                const float* wo_norm2, float epsilon, float* scores, cudaStream_t st);

// Quantised cache (FP8 E4M3 codes with scales): key codes widened to bf16 (exact), the weighting on value codes
// with one scale per token, and the gather of code rows with their value scales.
ea_status ea_launch_dequant_k(const ea_ctx* ctx, const ea_shape& s, const uint8_t* k_q8, __nv_bfloat16* k_codes,
                              cudaStream_t st);
ea_status ea_launch_finalize_q8(const ea_ctx* ctx, const ea_shape& s, const float* logits, const float* lse,
                                const uint8_t* v_q8, const float* v_scale, float epsilon, float* scores,
                                cudaStream_t st);
ea_status ea_launch_gather_q8(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* kept_idx,
                              const uint8_t* k_q8, const uint8_t* v_q8, const float* v_scale, uint8_t* k_out,
                              uint8_t* v_out, float* v_scale_out, cudaStream_t st);

ea_status ea_launch_select(const ea_ctx* ctx, const ea_shape& s, const float* scores, int n_kept,
                           int32_t* kept_idx, cudaStream_t st);

// Compaction inside the cache buffers: the kept rows of every head move to the front of its range.
// (codes: rows of head_dim one-byte codes instead of bf16)
ea_status ea_launch_compact_inplace(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* kept_idx,
                                    void* k, void* v, cudaStream_t st, bool codes = false);

// Unordered variant: kept rows beyond n_kept fill the evicted positions below it; `sel` ascending kept positions
// (scratch), `where` the original row at each position afterwards.
ea_status ea_launch_compact_fill(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* sel,
                                 int32_t* where, void* k, void* v, cudaStream_t st, bool codes = false);

// Head-adaptive eviction: per-head counts and offsets from one radix search over the unit's scores,
// then the per-head selection with those counts and a gather through the offsets.
size_t ea_adaptive_ws_bytes(const ea_shape& s);
ea_status ea_launch_select_adaptive(const ea_ctx* ctx, const ea_shape& s, const float* scores, int n_kept,
                                    int n_floor, void* ws, int32_t* kept_idx, int32_t* head_offsets,
                                    cudaStream_t st);
ea_status ea_launch_gather_adaptive(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* kept_idx,
                                    const int32_t* head_offsets, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                    __nv_bfloat16* k_out, __nv_bfloat16* v_out, cudaStream_t st);

ea_status ea_launch_gather(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* kept_idx,
                           const __nv_bfloat16* k, const __nv_bfloat16* v, __nv_bfloat16* k_out,
                           __nv_bfloat16* v_out, cudaStream_t st);
