/*
 * ea.h - C ABI of the Expected Attention KV-cache scoring and pruning library
 * for NVIDIA B200 (sm_100a).
 *
 * The library implements the compression routine of the Expected Attention
 * paper (Sec. 2.2, "Expected Attention: Estimating Attention From Future
 * Queries"; its compress() pseudo-code) as three asynchronous calls:
 *
 *   ea_query_stats     window queries -> position-averaged Gaussian (Eq. 5, 6)
 *   ea_score           closed-form expected attention of every cached key,
 *                      softmax over positions, GQA reduction, value-norm
 *                      weighting (Eq. 7, 8, 9)
 *   ea_select_compact  keep the n_kept highest-scoring pairs per KV head and
 *                      gather their K/V rows (the "Compression with Expected
 *                      Attention" paragraph)
 *
 * Conventions
 *   - One "unit" is one (layer, batch element).  A call handles n_units units
 *     that share every size; units, and the KV heads inside them, are
 *     independent problems.
 *   - Query head h reads KV head h / G, G = n_q_heads / n_kv_heads.
 *   - All data pointers are DEVICE pointers on the context's device unless a
 *     comment says HOST.  Tensors are dense, row-major, innermost index last.
 *     bf16 tensors are passed as const void* / void*.
 *   - The caller owns every data buffer.  The library never allocates, frees
 *     or keeps them; the only memory it owns is the context's workspace.
 *   - Calls enqueue work on cuda_stream (a cudaStream_t passed as void*; NULL
 *     is the default stream) and return without synchronising.  Work of one
 *     context must be ordered on one stream at a time (the workspace is
 *     shared between calls).
 *   - Errors that the host can detect are returned before anything is
 *     launched.  No call aborts, throws or traps the device.  A device-side
 *     wait that runs out of its iteration budget records
 *     EA_ERR_DEVICE_TIMEOUT, which ea_sync_status reports.
 *   - n_units * n_q_heads <= 65535 per call (EA_ERR_UNSUPPORTED beyond: split
 *     the units over several calls).
 *   - There is no CPU fallback: on a machine without an sm_100 GPU ea_create
 *     fails with EA_ERR_NOT_SM100 or EA_ERR_CUDA.
 */
#ifndef EA_H_
#define EA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum ea_status {
    EA_OK = 0,
    EA_ERR_INVALID_ARG = 1,    /* NULL pointer, bad size, misaligned buffer            */
    EA_ERR_UNSUPPORTED = 2,    /* head_dim or mode not implemented                     */
    EA_ERR_WORKSPACE = 3,      /* context workspace smaller than ea_workspace_bytes    */
    EA_ERR_CUDA = 4,           /* a CUDA runtime call failed                           */
    EA_ERR_NOT_SM100 = 5,      /* device is not compute capability 10.x                */
    EA_ERR_DEVICE_TIMEOUT = 6  /* a bounded device-side wait gave up                   */
} ea_status;

/* RoPE channel pairing used when the rotation is averaged (Eq. 6). */
enum { EA_ROPE_HALF_SPLIT = 0,   /* channel m pairs with m + d/2 (default)             */
       EA_ROPE_INTERLEAVED = 1 };/* channel 2m pairs with 2m + 1                       */
/* How the G query heads that share a KV head are combined (the paper only says
 * the analysis "extends to GQA"). */
enum { EA_GROUP_MEAN_PROB = 0,   /* softmax per query head, mean over the group (default) */
       EA_GROUP_SUM_PROB = 1,    /* softmax per query head, sum over the group            */
       EA_GROUP_MEAN_LOGIT = 2 };/* mean of the log-scores over the group, one softmax    */
/* Covariance normaliser. */
enum { EA_COV_POPULATION = 0,    /* 1/W (Gaussian maximum likelihood, default)         */
       EA_COV_SAMPLE = 1 };      /* 1/(W-1)                                            */

typedef struct ea_shape {
    int32_t n_units;     /* independent problems in this call: layers * batch          */
    int32_t n_q_heads;   /* Hq                                                         */
    int32_t n_kv_heads;  /* Hkv, divides Hq                                            */
    int32_t head_dim;    /* d: 64, 128 or 256                                          */
    int32_t n_keys;      /* n: cached keys per KV head (same for every unit)           */
    int32_t window;      /* W: window queries per query head                           */
    int32_t rope_layout; /* EA_ROPE_*                                                  */
    int32_t group_mode;  /* EA_GROUP_*                                                 */
    int32_t cov_norm;    /* EA_COV_*                                                   */
    int32_t kv_capacity; /* rows per KV head in the K/V BUFFERS when the cache lives in a
                            larger, fixed buffer (streaming decode): head g of unit u starts
                            at row (u * Hkv + g) * kv_capacity and its first n_keys rows are
                            the cache.  0 = dense (kv_capacity = n_keys).  Must be 0 or
                            >= n_keys.  Scores, log-scores and kept indices stay dense in
                            n_keys; gathered outputs (k_out, v_out) are dense in n_kept.   */
} ea_shape;

typedef struct ea_ctx ea_ctx;   /* opaque; owns its workspace and a status word */

/* Library version string, e.g. "ea-b200 0.2". */
const char* ea_version(void);
const char* ea_status_string(ea_status s);
/*
 * Which CUDA runtime call was behind the calling thread's most recent
 * EA_ERR_CUDA: "<error name> (<description>) at <source file>:<line>", or ""
 * if there has been none.  The string belongs to the library and is
 * overwritten by the thread's next failing call.
 */
const char* ea_last_cuda_error(void);

/*
 * Bytes of workspace the three calls need for this shape (the maximum over the
 * calls; they reuse it).  HOST-only arithmetic, no CUDA call.
 */
ea_status ea_workspace_bytes(const ea_shape* shape, size_t* out_bytes);

/*
 * n_kept = int(n_keys * (1 - compression_ratio)) as the paper's pseudo-code
 * computes it: product in double, truncated, clamped to [0, n_keys].  HOST-only.
 */
int64_t ea_n_kept(int64_t n_keys, double compression_ratio);

/*
 * Create a context on CUDA device `device` with a workspace of
 * workspace_bytes (allocated once here with cudaMalloc; 0 is allowed and can
 * only serve shapes that need none).  May synchronise.  Fails with
 * EA_ERR_NOT_SM100 unless the device has compute capability 10.x.
 */
ea_status ea_create(ea_ctx** out_ctx, int device, size_t workspace_bytes);
/* Frees the workspace.  The caller must have synchronised the streams used. */
ea_status ea_destroy(ea_ctx* ctx);

/*
 * Query statistics with the rotary embedding averaged over the future
 * positions (Eq. 5 and Eq. 6, queries given directly):
 *   mu      = (1/W) sum_w u_w                  per query head
 *   Sigma   = (1/N) sum_w (u_w-mu)(u_w-mu)^T   N = W or W-1 (cov_norm)
 *   R_bar   = (1/T) sum_{p=pos_next}^{pos_next+T-1} R_p,  R_p the RoPE rotation
 *             at position p with theta_m = rope_base^(-2m/d)
 *   mu_bar  = R_bar mu,   sigma_bar = R_bar Sigma R_bar^T
 *
 * q_win     bf16 [n_units, Hq, W, d]  PRE-RoPE window queries, 16-byte aligned
 * pos_next  int64 [n_units] DEVICE: 0-based position of the first future token
 *           of each unit (n_keys for a prefill cache holding positions 0..n-1)
 * n_future  T >= 1
 * mu_bar    fp32 [n_units, Hq, d]      (output)
 * sigma_bar fp32 [n_units, Hq, d, d]   (output, symmetric)
 * shape->n_keys is ignored.  Requires W >= 1 (W >= 2 for EA_COV_SAMPLE).
 */
ea_status ea_query_stats(ea_ctx* ctx, const ea_shape* shape, const void* q_win,
                         const int64_t* pos_next, int32_t n_future, double rope_base,
                         float* mu_bar, float* sigma_bar, void* cuda_stream);

/*
 * ea_query_stats for callers that cannot allocate device memory (the paper has
 * no counterpart: this is a packaging variant, the arithmetic and the outputs
 * are those of ea_query_stats).
 *
 * Who needs it: code that runs where cudaMalloc is off limits - inside a
 * serving loop whose memory is fully handed to a caching allocator, in a
 * plugin whose host forbids driver allocations after start-up, or on a
 * latency path where an allocation's implicit device synchronisation is not
 * acceptable.  ea_create allocates (the workspace and a pinned status word),
 * so this call takes no context: it uses the CURRENT device and only launches
 * kernels on cuda_stream.
 *
 * The one piece of scratch the statistics need, the averaged-rotation
 * coefficients (one fp32 cos/sin pair per unit and channel pair), lives in a
 * fixed array inside the library: EA_STATIC_MAX_ROPE_PAIRS pairs, 128 KiB,
 * held by every GPU that loads the library until the process exits.  A shape
 * with n_units * head_dim / 2 > EA_STATIC_MAX_ROPE_PAIRS is refused with
 * EA_ERR_WORKSPACE before anything is launched (split the units over several
 * calls on the same stream).
 *
 * The first call on each device looks up the array's device address (no
 * allocation, but a runtime query): make that first call before starting any
 * stream capture.  All calls on a device share the array.  Each call rewrites
 * every coefficient it later reads, so nothing left by an earlier call can
 * leak into the result and nothing needs clearing; but two calls whose kernels
 * overlap on the GPU (different streams, no ordering between them) race on
 * it.  Order them on one stream or with events.
 *
 * Arguments as for ea_query_stats (pos_next is a DEVICE pointer); n_keys,
 * n_kv_heads and group_mode of the shape are ignored.
 */
#define EA_STATIC_MAX_ROPE_PAIRS 16384
ea_status ea_query_stats_static(const ea_shape* shape, const void* q_win, const int64_t* pos_next,
                                int32_t n_future, double rope_base, float* mu_bar, float* sigma_bar,
                                void* cuda_stream);

/*
 * The same statistics from buffered hidden states (Eq. 5 as the paper writes
 * it: h ~ N(mu_h, Sigma_h), q = W_Q h, so mu = W_Q mu_h and
 * Sigma = W_Q Sigma_h W_Q^T per query head; the decoding set-up keeps a
 * buffer of the last hidden states for this).  The library projects the W
 * buffered rows (Q = H W_Q^T on the tensor cores, fp32) and takes the mean and
 * covariance of the projected rows, which are those two expressions exactly;
 * the d_model x d_model covariance is never formed.  Then Eq. 6 as in
 * ea_query_stats.
 *
 * hidden     bf16 [n_units, W, d_model]  the inputs of the query projection
 *            (i.e. after the layer's input norm), W = shape->window <= 512
 * w_q        bf16 [n_weight_sets, Hq * d, d_model]  query projections; row
 *            j * d + c of a set is row c of W_Q of head j.  Units are taken
 *            set-major: unit u uses set u / (n_units / n_weight_sets)
 *            (n_units = layers * batch with one set per layer).
 * d_model    a multiple of 8
 * q_scratch  fp32 [n_units, Hq, W, d]  caller-owned scratch; holds the
 *            projected window queries on return
 * the other arguments as for ea_query_stats.
 * EA_ERR_UNSUPPORTED for W > 512; EA_ERR_INVALID_ARG for a bad d_model or
 * n_weight_sets that does not divide n_units.
 */
ea_status ea_query_stats_hidden(ea_ctx* ctx, const ea_shape* shape, const void* hidden,
                                const void* w_q, int32_t d_model, int32_t n_weight_sets,
                                float* q_scratch, const int64_t* pos_next, int32_t n_future,
                                double rope_base, float* mu_bar, float* sigma_bar,
                                void* cuda_stream);

/*
 * Contribution score of every cached pair (Eq. 7, 8, 9 with ||v|| in place of
 * ||W_o v||, as the paper's implementation note states):
 *   s_{h,i}   = mu_bar_h . k_i / sqrt(d) + k_i^T sigma_bar_h k_i / (2d)
 *   a_{h,i}   = exp(s_{h,i} - logsumexp_i s_{h,.})          softmax over the n keys
 *   a_{g,i}   = group reduction of a_{h,i} over the G heads of KV head g (group_mode)
 *   score_{g,i} = (a_{g,i} + epsilon) * ||v_{g,i}||_2
 * Everything stays in the log domain until the softmax, so outlier-heavy
 * activations do not overflow.
 *
 * k, v       bf16 [n_units, Hkv, n, d]; K is POST-RoPE; 16-byte aligned
 * mu_bar     fp32 [n_units, Hq, d];  sigma_bar fp32 [n_units, Hq, d, d]
 * scores     fp32 [n_units, Hkv, n]  (output)
 * logits_opt fp32 [n_units, Hq, n] or NULL: when given, receives s_{h,i}
 * shape->window is ignored.  n_keys == 0 or n_units == 0 is a no-op.
 */
ea_status ea_score(ea_ctx* ctx, const ea_shape* shape, const void* k, const void* v,
                   const float* mu_bar, const float* sigma_bar, float epsilon, float* scores,
                   float* logits_opt, void* cuda_stream);

/*
 * Contribution scores with the output projection (Eq. 9 as written:
 * (a_hat + epsilon) * ||W_o v||; the paper's experiments drop W_o, see
 * ea_score).  Query head h multiplies the value it reads by its own slice
 * W_o^h = W_o[:, h*d : (h+1)*d], so per query head
 *   c_{h,i} = (a_hat_{h,i} + epsilon) * ||W_o^h v_{g,i}||_2,
 * reduced over the G heads of KV head g like the attention itself (mean for
 * EA_GROUP_MEAN_PROB, sum for EA_GROUP_SUM_PROB; EA_GROUP_MEAN_LOGIT has no
 * per-head attention: EA_ERR_UNSUPPORTED).  ||W_o^h v||^2 = v^T M_h v with the
 * Gram matrix M_h = W_o^h^T W_o^h, which ea_wo_gram computes once per model;
 * the quadratic form runs on the same tensor-core kernel as Eq. 7, with the
 * value rows in place of the keys.
 *
 * ea_wo_gram
 *   w_o      bf16 [n_weight_sets, d_model, Hq * d]  output projections (row =
 *            output channel), 16-byte aligned
 *   wo_gram  fp32 [n_weight_sets, Hq, d, d]  (output)
 * ea_score_wo: the arguments of ea_score, plus
 *   wo_gram, n_weight_sets   as above; units are set-major: unit u uses set
 *            u / (n_units / n_weight_sets); n_weight_sets must divide n_units
 *   wo_scratch fp32 [n_units, Hq, n]  caller-owned scratch; holds
 *            ||W_o^h v_i||^2 on return
 */
ea_status ea_wo_gram(ea_ctx* ctx, const void* w_o, int32_t d_model, int32_t n_weight_sets,
                     int32_t n_q_heads, int32_t head_dim, float* wo_gram, void* cuda_stream);
ea_status ea_score_wo(ea_ctx* ctx, const ea_shape* shape, const void* k, const void* v,
                      const float* mu_bar, const float* sigma_bar, const float* wo_gram,
                      int32_t n_weight_sets, float epsilon, float* wo_scratch, float* scores,
                      float* logits_opt, void* cuda_stream);

/*
 * The same scores on a quantised cache.  The paper calls quantisation
 * orthogonal to eviction and combinable with it (Related Works,
 * "Quantization") and fixes no format; this library's reading: keys and values
 * are FP8 E4M3 codes (1 sign, 4 exponent bits with bias 7, 3 mantissa bits, no
 * infinities, largest finite value 448) with fp32 scales,
 *   k[u,g,i,c] = decode(k_q8[u,g,i,c]) * k_scale[u,g,c]     one scale per channel
 *   v[u,g,i,c] = decode(v_q8[u,g,i,c]) * v_scale[u,g,i]     one scale per token
 * and the scores are Eq. 7, 8, 9 of ea_score on these k, v.  The key scales
 * are folded into mu_bar and sigma_bar (mu.k = (s*mu).x and
 * k^T Sigma k = x^T diag(s) Sigma diag(s) x for the code row x), so the tensor-
 * core kernel runs on the codes, widened to bf16 without rounding; the value
 * norm is v_scale_i ||x_i||.
 *
 * k_q8, v_q8  uint8 [n_units, Hkv, cap, d] E4M3 codes, 16-byte aligned; cap = kv_capacity
 *             (n_keys when that is 0): the first n_keys rows of a head's range are its cache
 * k_scale     fp32 [n_units, Hkv, d];   v_scale  fp32 [n_units, Hkv, cap]
 * k_scratch   bf16 [n_units, Hkv, cap, d]  caller-owned scratch for the widened key
 *             codes.  Needed, and written, only where the tensor-core kernel,
 *             which widens the codes itself, does not take the shape (fewer
 *             keys than one tile: 128, or 256 at head_dim 256; query groups of
 *             more than 16 head subsets); ea_score_q8_scratch_bytes says how
 *             many bytes that is, 0 meaning that k_scratch may be NULL
 * the other arguments as for ea_score.
 */
ea_status ea_score_q8(ea_ctx* ctx, const ea_shape* shape, const void* k_q8, const float* k_scale,
                      const void* v_q8, const float* v_scale, const float* mu_bar,
                      const float* sigma_bar, float epsilon, void* k_scratch, float* scores,
                      float* logits_opt, void* cuda_stream);
/* Host only: bytes of k_scratch that ea_score_q8 needs for this shape (0: none). */
ea_status ea_score_q8_scratch_bytes(const ea_shape* shape, size_t* bytes);
/*
 * ea_select_compact on a quantised cache: the same selection, then the kept
 * code rows and the value scales of their tokens are gathered (the key scales
 * belong to the channels and stay as they are).  The source may sit in a
 * larger buffer (kv_capacity); the outputs are dense.
 * k_out, v_out  uint8 [n_units, Hkv, n_kept, d];  v_scale_out fp32 [n_units, Hkv, n_kept]
 */
ea_status ea_select_compact_q8(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                               int32_t n_kept, const void* k_q8, const void* v_q8,
                               const float* v_scale, int32_t* kept_idx, void* k_out, void* v_out,
                               float* v_scale_out, void* cuda_stream);
/*
 * ea_select_compact_adaptive (head-adaptive eviction, same arguments and
 * errors) on a quantised cache: ragged outputs k_out, v_out uint8
 * [n_units, Hkv * n_kept, d] and v_scale_out fp32 [n_units, Hkv * n_kept],
 * head g of unit u owning the rows head_offsets[u, g] .. head_offsets[u, g + 1].
 * The outputs are always gathered (all three required when n_kept > 0).
 */
ea_status ea_select_compact_adaptive_q8(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                                        int32_t n_kept, int32_t n_floor, const void* k_q8,
                                        const void* v_q8, const float* v_scale, int32_t* kept_idx,
                                        int32_t* head_offsets, void* k_out, void* v_out,
                                        float* v_scale_out, void* cuda_stream);
/*
 * Streaming decode on a quantised cache (the decoding set-up of Sec. 4 with
 * the format above): the two calls that let one buffer of codes live through
 * consecutive compression events, beside ea_window_push / ea_query_stats_ring
 * and ea_score_q8 with kv_capacity.
 *
 * ea_cache_append_q8: n_new code rows per head, k_new / v_new uint8
 * [n_units, Hkv, n_new, d] with their value scales v_scale_new fp32
 * [n_units, Hkv, n_new], go behind the shape->n_keys rows each head holds;
 * the new key codes are codes against the cache's own key scales.
 * n_keys + n_new > capacity: EA_ERR_INVALID_ARG.  Device pointers, 16-byte
 * aligned codes; asynchronous on cuda_stream.
 *
 * ea_select_compact_inplace_q8: ea_select_compact_inplace (unordered == 0:
 * kept rows move to the front of the head's range in ascending order of
 * position, kept_idx ascending) or ea_select_compact_inplace_unordered
 * (unordered != 0: kept rows beyond n_kept fill the evicted positions below
 * it; kept_idx[j] = the original row now at position j; needs the context's
 * workspace and 2 * n_kept * 4 bytes <= 200 KiB) on code rows; the value
 * scales move with their rows.  k_q8 and v_q8 must not overlap.
 */
ea_status ea_cache_append_q8(ea_ctx* ctx, const ea_shape* shape, void* k_q8, void* v_q8, float* v_scale,
                             const void* k_new, const void* v_new, const float* v_scale_new,
                             int32_t n_new, void* cuda_stream);
ea_status ea_select_compact_inplace_q8(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                                       int32_t n_kept, void* k_q8, void* v_q8, float* v_scale,
                                       int32_t* kept_idx, int32_t unordered, void* cuda_stream);

/*
 * Eviction and compaction: per (unit, KV head) keep the n_kept pairs with the
 * highest score; among equal scores the lowest index wins; kept indices are
 * emitted in ascending order (the cache keeps its temporal order) and the
 * K/V rows are gathered in that order.
 *
 * scores    fp32 [n_units, Hkv, n] (any finite values; -0 is treated as +0)
 * n_kept    0 <= n_kept <= n_keys (EA_ERR_INVALID_ARG otherwise)
 * k, v      bf16 [n_units, Hkv, n, d], 16-byte aligned
 * kept_idx  int32 [n_units, Hkv, n_kept]        (output)
 * k_out,v_out bf16 [n_units, Hkv, n_kept, d]    (output; must not overlap k, v)
 *           k_out/v_out may both be NULL to skip the gather (indices only).
 */
ea_status ea_select_compact(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                            int32_t n_kept, const void* k, const void* v, int32_t* kept_idx,
                            void* k_out, void* v_out, void* cuda_stream);

/*
 * Eviction with compaction inside the cache (for a cache that lives in a
 * fixed buffer and is compressed periodically while decoding, as in the
 * paper's decoding set-up): the selection of ea_select_compact, then the kept
 * rows of every head are moved, in order, to the front of that head's range:
 *   k[u, g, j, :] <- k[u, g, kept_idx[u, g, j], :]   for j < n_kept, same for v.
 * Rows n_kept .. n-1 of each head keep whatever they held (the caller's cache
 * length becomes n_kept; new pairs are appended from there).  kept_idx still
 * refers to the positions before the call.
 *
 * k, v      bf16 [n_units, Hkv, n, d] (rows per head: kv_capacity if set), 16-byte
 *           aligned, modified in place; two distinct buffers
 * kept_idx  int32 [n_units, Hkv, n_kept]  (output)
 * The call records only stream work and no allocation, so a sequence of
 * ea_query_stats / ea_score / ea_select_compact_inplace can be captured into
 * a CUDA graph and replayed for every compression event of the same shape.
 */
ea_status ea_select_compact_inplace(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                                    int32_t n_kept, void* k, void* v, int32_t* kept_idx,
                                    void* cuda_stream);

/*
 * The same eviction without the temporal order (the paper has no counterpart:
 * attention does not depend on the order of the cached pairs, and post-RoPE
 * keys carry their positions).  Kept rows below n_kept stay where they are; the
 * kept rows at or beyond n_kept move, in ascending order, into the evicted
 * positions below n_kept, in ascending order.  In a stream that appends a few
 * hundred pairs per event to a cache of thousands this moves only about as many
 * rows as were appended, where the ordered compaction moves almost every row.
 * kept_idx[u, g, j] is the position, before the call, of the row that sits at j
 * afterwards: the same SET as ea_select_compact_inplace returns, in the new
 * physical order (not ascending).  n_kept <= 25600 (EA_ERR_UNSUPPORTED beyond);
 * needs the context's workspace (EA_ERR_WORKSPACE if smaller than
 * ea_workspace_bytes(shape)).  Arguments as for ea_select_compact_inplace.
 */
ea_status ea_select_compact_inplace_unordered(ea_ctx* ctx, const ea_shape* shape,
                                              const float* scores, int32_t n_kept, void* k, void* v,
                                              int32_t* kept_idx, void* cuda_stream);

/*
 * Carried value norms (streaming decode, Sec. 4's set-up; the paper has no
 * counterpart).  ||v_i|| of Eq. 9 does not change while pair i stays in the
 * cache, so a cache that lives through consecutive compression events can
 * carry the norms with it: v_norm fp32 [n_units, Hkv, capacity] (capacity =
 * kv_capacity, or n_keys when that is 0), entry i of a head's range = ||v||
 * of the head's row i.  Scoring then reads 4 bytes per cached pair in place
 * of its value row.
 *
 * ea_value_norms: v_norm[u, g, i] = ||v[u, g, i, :]|| (fp32 accumulation) for
 * first_row <= i < first_row + n_rows of every head; the rows need not lie
 * below n_keys (first_row + n_rows <= capacity, else EA_ERR_INVALID_ARG).
 * After ea_cache_append: first_row = the old n_keys, n_rows = n_new.
 *
 * ea_score_vnorm: ea_score with v_norm in place of v; every other argument,
 * the fused form with NULL statistics included, as for ea_score.  The scores
 * agree with ea_score's to fp32 rounding of the sum of squares.
 *
 * ea_carry_f32_inplace: values[u, g, j] <- values[u, g, kept_idx[u, g, j]] for
 * j < n_kept, for a per-token fp32 array [n_units, Hkv, capacity] such as
 * v_norm: what ea_select_compact_inplace or
 * ea_select_compact_inplace_unordered did to the rows, given the kept_idx that
 * call returned (both satisfy kept_idx[j] >= j, which the move relies on).
 * Device pointers; asynchronous on cuda_stream.
 */
ea_status ea_value_norms(ea_ctx* ctx, const ea_shape* shape, const void* v, int32_t first_row,
                         int32_t n_rows, float* v_norm, void* cuda_stream);
ea_status ea_score_vnorm(ea_ctx* ctx, const ea_shape* shape, const void* k, const float* v_norm,
                         const float* mu_bar, const float* sigma_bar, float epsilon, float* scores,
                         float* logits_opt, void* cuda_stream);
ea_status ea_carry_f32_inplace(ea_ctx* ctx, const ea_shape* shape, const int32_t* kept_idx,
                               int32_t n_kept, float* values, void* cuda_stream);

/*
 * Streaming decode: one cache buffer and one window buffer carried through
 * consecutive compression events (the decoding set-up of the "Implementation
 * details" paragraph: a buffer of the most recent 128 states, compression
 * every 512 generated tokens down to a fixed budget).
 *
 * The cache of a head lives in a fixed range of kv_capacity rows (see
 * ea_shape) of which the first n_keys are valid.  One event is
 *   ea_cache_append            n_keys -> n_keys + n_new rows per head
 *   ea_window_push             the queries generated since the last event
 *   ea_query_stats_ring        statistics of what the window ring holds
 *   ea_score                   on the shape with the new n_keys
 *   ea_select_compact_inplace  back to the budget, kept rows moved to the front
 * after which the caller's n_keys is n_kept.  All five only enqueue stream
 * work on device-resident state, so an event of a given shape can be captured
 * into a CUDA graph once and replayed.
 *
 * ea_cache_append
 *   k, v          bf16 [n_units, Hkv, kv_capacity, d], modified in place: rows
 *                 n_keys .. n_keys + n_new - 1 of every head receive the new pairs
 *   k_new, v_new  bf16 [n_units, Hkv, n_new, d] (K POST-RoPE at its absolute position)
 *   n_keys + n_new <= kv_capacity, else EA_ERR_INVALID_ARG
 * ea_window_push
 *   q_ring        bf16 [n_units, Hq, W, d], W = shape->window: a ring per query head
 *   ring_pushed   int64 [n_units] DEVICE: rows pushed so far per unit (start at 0);
 *                 row j of this call goes to ring row (ring_pushed + j) mod W, then
 *                 the counters advance by n_new.  The window is the last
 *                 min(ring_pushed, W) rows pushed.
 *   q_new         bf16 [n_units, Hq, n_new, d] PRE-RoPE queries, oldest first
 * ea_query_stats_ring
 *   ea_query_stats over the rows the ring holds: min(ring_pushed[u], W) of them
 *   (a partly filled ring is read by its first rows, a wrapped one as it lies:
 *   mean and covariance do not depend on the order).  A unit with fewer than
 *   one row (two for EA_COV_SAMPLE) gets mu_bar = 0, sigma_bar = 0.
 */
ea_status ea_cache_append(ea_ctx* ctx, const ea_shape* shape, void* k, void* v, const void* k_new,
                          const void* v_new, int32_t n_new, void* cuda_stream);
ea_status ea_window_push(ea_ctx* ctx, const ea_shape* shape, void* q_ring, int64_t* ring_pushed,
                         const void* q_new, int32_t n_new, void* cuda_stream);
ea_status ea_query_stats_ring(ea_ctx* ctx, const ea_shape* shape, const void* q_ring,
                              const int64_t* ring_pushed, const int64_t* pos_next, int32_t n_future,
                              double rope_base, float* mu_bar, float* sigma_bar, void* cuda_stream);

/*
 * Head-adaptive eviction and compaction (the "Head-Adaptive Compression"
 * paragraph of Sec. 2.2: the per-layer budget allocation of Ada-KV, so that
 * heads whose pairs matter more retain more of them).  The paper prints no
 * formula; the rule is the published one with its safeguard:
 *
 *   A unit (one layer of one sequence) has a budget of Hkv * n_kept pairs.
 *   1. Every head keeps its n_floor best pairs (score descending, index
 *      ascending).
 *   2. The other Hkv * (n_kept - n_floor) places go to the best pairs not yet
 *      kept, over all heads of the unit (score descending, then head
 *      ascending, then index ascending).
 *   3. The kept indices of a head are emitted ascending, heads one after the
 *      other: kept_idx[u][head_offsets[u][g] .. head_offsets[u][g+1]) belongs
 *      to head g, and K/V rows are gathered in that order.
 *
 * n_floor == n_kept gives the result of ea_select_compact; n_floor == 0 is
 * one top-(Hkv * n_kept) over the unit.  ea_n_floor gives the safeguard share
 * floor(safeguard * n_kept) (the published default safeguard is 0.2).
 *
 * scores       fp32 [n_units, Hkv, n] (any finite values; -0 is treated as +0)
 * n_kept       0 <= n_kept <= n_keys; n_floor: 0 <= n_floor <= n_kept;
 *              Hkv * n_kept < 2^31 (EA_ERR_INVALID_ARG otherwise)
 * k, v         bf16 [n_units, Hkv, n, d], 16-byte aligned
 * kept_idx     int32 [n_units, Hkv * n_kept]       (output; key index within its head)
 * head_offsets int32 [n_units, Hkv + 1]            (output; first is 0, last is Hkv * n_kept)
 * k_out,v_out  bf16 [n_units, Hkv * n_kept, d]     (output; must not overlap k, v)
 *              k_out/v_out may both be NULL to skip the gather.
 * Uses the context's workspace (EA_ERR_WORKSPACE if smaller than
 * ea_workspace_bytes(shape)).
 */
ea_status ea_select_compact_adaptive(ea_ctx* ctx, const ea_shape* shape, const float* scores,
                                     int32_t n_kept, int32_t n_floor, const void* k, const void* v,
                                     int32_t* kept_idx, int32_t* head_offsets, void* k_out,
                                     void* v_out, void* cuda_stream);

/* floor(safeguard * n_kept) evaluated in double, clamped to [0, n_kept]. */
int64_t ea_n_floor(int64_t n_kept, double safeguard);

/*
 * Limits the persistent log-score kernel of this context (Eq. 7; one CTA per SM,
 * each taking the SM's whole register file and shared memory) to n_sms SMs,
 * so that work launched beside it - another context's memory-bound passes, a
 * decode step of the serving engine - finds the other SMs free instead of
 * queueing behind it (the paper has no counterpart).  n_sms = 0 restores the
 * default, every SM of the device.  32 <= n_sms <= SM count, else
 * EA_ERR_INVALID_ARG.  Takes effect from the next ea_score / ea_score_wo.
 */
ea_status ea_set_sm_budget(ea_ctx* ctx, int32_t n_sms);

/*
 * Fused statistics (the paper has no counterpart; a shortcut for the streaming
 * path, where a compression event scores a few thousand keys for thousands of
 * query heads and preparing the tensor-core operand from sigma_bar is a
 * noticeable part of it).  With on != 0, ea_query_stats and
 * ea_query_stats_ring also write, straight from their accumulators, the bf16
 * operand that ea_score's tensor-core kernel would otherwise build from
 * mu_bar and sigma_bar, into the context's workspace; a following
 *     ea_score(ctx, shape, k, v, NULL, NULL, ...)
 * on the SAME context with the SAME shape (every field but `window`) uses it
 * and needs neither array.  In this mode sigma_bar may be NULL in the statistics
 * call (mu_bar is still written).  The scores are bit for bit those of the
 * two-step path.  Conditions: head_dim 64 or 128, n_keys >= 128, group mode
 * not EA_GROUP_MEAN_LOGIT, workspace of ea_workspace_bytes(shape); otherwise
 * the statistics call behaves as without the flag (and then needs sigma_bar),
 * and ea_score with NULL statistics returns EA_ERR_INVALID_ARG.  Any later
 * statistics call of the context replaces the operand; a scoring call that is
 * given statistics (ea_score with sigma_bar, ea_score_wo, ea_score_q8) builds
 * its own operand in the same place, after which ea_score with NULL statistics
 * is refused until the next statistics call.
 */
ea_status ea_set_fused_stats(ea_ctx* ctx, int32_t on);

/*
 * Runs the value-norm pass of ea_score (the ||v|| of Eq. 9, which does not
 * depend on the log-scores) on n_sms SMs of its own, beside the tensor-bound
 * log-score kernel instead of after it (the paper has no counterpart): a
 * persistent kernel of n_sms CTAs streams V through bulk copies on a stream the
 * context owns, the log-score kernel takes the other SMs, and a light weighting
 * pass joins the two.  The scores are those of the default path up to the
 * rounding of one fp32 square root.  n_sms even, 0 <= n_sms <= SM count - 32
 * (EA_ERR_INVALID_ARG otherwise); 0 (the default) switches the side pass off.
 * The first call with n_sms > 0 creates the stream and two events: make it
 * outside a stream capture.  Applies to ea_score with the tensor-core path
 * (head_dim 64/128/256 and at least one tile of keys); other calls ignore it.
 */
ea_status ea_set_side_sms(ea_ctx* ctx, int32_t n_sms);

/*
 * Synchronises cuda_stream and returns the device-side status recorded since
 * the last call of this function (EA_OK, EA_ERR_DEVICE_TIMEOUT, or
 * EA_ERR_CUDA if the stream reports an error), then clears it.
 */
ea_status ea_sync_status(ea_ctx* ctx, void* cuda_stream);

/*
 * Self-test of the device-timeout route (the paper has no counterpart).  Every
 * wait inside the library's kernels is bounded; one that gives up raises the
 * context's status word, which ea_sync_status reports as
 * EA_ERR_DEVICE_TIMEOUT.  This call launches a one-thread kernel that waits,
 * with the same bounded wait and a limit of limit_us microseconds
 * (1 <= limit_us <= 1000, EA_ERR_INVALID_ARG otherwise), on a barrier that
 * nothing signals, so the wait runs out by construction; no copy is in flight
 * and nothing is held, the kernel returns by itself and the context stays
 * usable.  After it, ea_sync_status returns EA_ERR_DEVICE_TIMEOUT once and
 * EA_OK from then on.  The production waits keep their own limit (2 s: far
 * longer than any healthy wait, also under a profiler's replay or on a GPU
 * shared with other processes; a genuine stall surfaces the same way).
 */
ea_status ea_selftest_wait_timeout(ea_ctx* ctx, int32_t limit_us, void* cuda_stream);

/*
 * The whole routine on HOST buffers: compress(queries, keys, values) ->
 * (kept indices, keys[idx], values[idx]) as in the paper's pseudo-code, for
 * callers whose cache lives in host memory.  Units are processed in chunks of
 * units_per_chunk; each chunk is copied to the device, run through
 * ea_query_stats, ea_score and ea_select_compact, and its results copied
 * back, with the copies of neighbouring chunks overlapping the kernels (two
 * staging buffers, two internal copy streams).  Every pointer here is a HOST
 * pointer; pinned memory (cudaHostAlloc / cudaHostRegister) is needed for the
 * copies to overlap, pageable memory works but serialises.  The call returns
 * after enqueuing; the host buffers must stay valid and untouched until
 * cuda_stream has been synchronised (ea_sync_status does that).
 *
 * shape            sizes of the WHOLE problem (n_units = all units)
 * q_win,k,v        bf16 host arrays shaped as for the device calls
 * pos_next         int64 [n_units] host
 * kept_idx         int32 [n_units, Hkv, n_kept] host (output)
 * k_out, v_out     bf16 [n_units, Hkv, n_kept, d] host (output)
 * scores_opt       fp32 [n_units, Hkv, n] host or NULL (output)
 * The context's workspace must hold ea_host_workspace_bytes(shape, n_kept,
 * units_per_chunk) bytes (staging for two chunks plus the kernels' workspace).
 */
ea_status ea_host_workspace_bytes(const ea_shape* shape, int32_t n_kept, int32_t units_per_chunk,
                                  size_t* out_bytes);
ea_status ea_compress_host(ea_ctx* ctx, const ea_shape* shape, const void* q_win, const void* k,
                           const void* v, const int64_t* pos_next, int32_t n_future,
                           double rope_base, float epsilon, int32_t n_kept, int32_t units_per_chunk,
                           int32_t* kept_idx, void* k_out, void* v_out, float* scores_opt,
                           void* cuda_stream);

/*
 * Instrumentation for benchmarks (the paper has no counterpart).  Between
 * ea_profile_begin and ea_profile_end the context counts every kernel it
 * launches and brackets each launch of the log-score kernel (Eq. 7, the
 * dominant kernel) with CUDA events on the caller's stream.  ea_profile_end
 * synchronises cuda_stream and reports the summed device time of those
 * launches in milliseconds, how many there were, and the total number of
 * kernel launches.  At most 4096 log-score launches are timed per window;
 * later ones are counted but not timed (timed_launches tells how many were).
 */
ea_status ea_profile_begin(ea_ctx* ctx);
ea_status ea_profile_end(ea_ctx* ctx, void* cuda_stream, double* score_kernel_ms,
                         int64_t* timed_launches, int64_t* total_kernel_launches);

#ifdef __cplusplus
}
#endif
#endif /* EA_H_ */
