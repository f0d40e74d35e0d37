// Log-scores s_{h,i} = mu_bar_h.k_i/sqrt(d) + k_i^T Sigma_bar_h k_i/(2d) (Eq. 7)
// on the fp32 CUDA cores.  Each warp owns 8 keys of one query head; lanes split
// the d columns of t = Sigma_bar k, so every Sigma_bar row is read once per
// 8 keys (coalesced, L2/L1 resident) and the key values come from shared
// memory as broadcasts.
#include "ea_internal.h"

namespace {

constexpr int kThreads = 256;
constexpr int kKeysPerWarp = 8;
constexpr int kKeysPerCta = (kThreads / 32) * kKeysPerWarp;   // 64

template <int D>
__global__ void __launch_bounds__(kThreads)
logits_simt_kernel(const __nv_bfloat16* __restrict__ k, const ea_quad_form form, int Hq, int Hkv, int n, int cap,
                   float* __restrict__ logits) {
    constexpr int CT = D / 32;
    __shared__ __nv_bfloat16 k_s[kKeysPerCta][D];

    const int uh = blockIdx.y;
    const int u = uh / Hq, h = uh % Hq, g = h / (Hq / Hkv);
    const int key0 = blockIdx.x * kKeysPerCta;
    const __nv_bfloat16* kk = k + ((size_t)u * Hkv + g) * (size_t)cap * D;
    const size_t set_head = (size_t)(u / form.units_per_set) * Hq + h;
    const float* S = form.quad + set_head * D * D;
    const float* mu = form.lin ? form.lin + set_head * D : nullptr;
    // per-channel scales of quantised rows, folded into the form as it is read
    const float* cs = form.ch_scale ? form.ch_scale + ((size_t)u * Hkv + g) * D : nullptr;
    float cs_r[CT];
#pragma unroll
    for (int j = 0; j < CT; ++j) cs_r[j] = cs ? cs[(threadIdx.x % 32) + 32 * j] : 1.f;

    for (int e = threadIdx.x; e < kKeysPerCta * D; e += kThreads) {
        int r = e / D, c = e % D;
        k_s[r][c] = (key0 + r < n) ? kk[(size_t)(key0 + r) * D + c] : __float2bfloat16(0.f);
    }
    __syncthreads();

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const __nv_bfloat16(*kw)[D] = &k_s[warp * kKeysPerWarp];
    float t[kKeysPerWarp][CT];
#pragma unroll
    for (int i = 0; i < kKeysPerWarp; ++i)
#pragma unroll
        for (int j = 0; j < CT; ++j) t[i][j] = 0.f;

    for (int a = 0; a < D; ++a) {
        float srow[CT];
#pragma unroll
        for (int j = 0; j < CT; ++j) srow[j] = S[(size_t)a * D + lane + 32 * j] * (cs ? cs[a] * cs_r[j] : 1.f);
#pragma unroll
        for (int i = 0; i < kKeysPerWarp; ++i) {
            const float ka = __bfloat162float(kw[i][a]);
#pragma unroll
            for (int j = 0; j < CT; ++j) t[i][j] = fmaf(ka, srow[j], t[i][j]);
        }
    }

    const float inv_sqrt_d = form.lin_scale;
    const float inv_2d = form.quad_scale;
    float mu_r[CT];
#pragma unroll
    for (int j = 0; j < CT; ++j) mu_r[j] = mu ? mu[lane + 32 * j] * inv_sqrt_d * cs_r[j] : 0.f;
#pragma unroll
    for (int i = 0; i < kKeysPerWarp; ++i) {
        float acc = 0.f;
#pragma unroll
        for (int j = 0; j < CT; ++j)
            acc = fmaf(__bfloat162float(kw[i][lane + 32 * j]), fmaf(t[i][j], inv_2d, mu_r[j]), acc);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
        const int key = key0 + warp * kKeysPerWarp + i;
        if (lane == 0 && key < n) logits[(size_t)uh * n + key] = acc;
    }
}

}  // namespace

ea_status ea_launch_logits_simt(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* k,
                                const ea_quad_form& form, float* logits, cudaStream_t st) {
    ea_count_launches(ctx, 1);
    cudaEvent_t stop = ea_profile_mark_start(ctx, st);
    dim3 grid((unsigned)((s.n_keys + kKeysPerCta - 1) / kKeysPerCta),
              (unsigned)(s.n_units * s.n_q_heads));
    switch (s.head_dim) {
        case 64:
            logits_simt_kernel<64><<<grid, kThreads, 0, st>>>(k, form, s.n_q_heads,
                                                             s.n_kv_heads, s.n_keys, ea_kv_cap(s), logits);
            break;
        case 128:
            logits_simt_kernel<128><<<grid, kThreads, 0, st>>>(k, form, s.n_q_heads,
                                                              s.n_kv_heads, s.n_keys, ea_kv_cap(s), logits);
            break;
        case 256: {
            auto kern = logits_simt_kernel<256>;
            kern<<<grid, kThreads, 0, st>>>(k, form, s.n_q_heads, s.n_kv_heads, s.n_keys, ea_kv_cap(s), logits);
            break;
        }
        default:
            return EA_ERR_UNSUPPORTED;
    }
    ea_profile_mark_stop(ctx, stop, st);
    return EA_CHECK_LAUNCH();
}
