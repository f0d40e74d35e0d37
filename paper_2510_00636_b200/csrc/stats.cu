// Query statistics with the rotary embedding averaged over future positions
// (Eq. 5 and Eq. 6 of the paper, window queries given directly).
//
// Kernel 1 (rope_coef_kernel): for each unit and rotation pair m, the mean of
// cos/sin(p * theta_m) over p = pos_next .. pos_next + T - 1, evaluated in fp64
// with the closed form of the geometric series
//   (1/T) sum_j e^{i theta (p+j)} = e^{i theta (p + (T-1)/2)} sin(T theta/2) / (T sin(theta/2)).
// Kernel 2 (stats_kernel): per query head, mu_bar = R_bar mu and
//   Sigma_bar = (1/N) sum_w x_w x_w^T,  x_w = R_bar (u_w - mu),
// which equals R_bar Sigma R_bar^T.  fp32 accumulation of bf16 inputs.
#include "ea_internal.h"

namespace {

__global__ void rope_coef_kernel(const int64_t* __restrict__ pos_next, int n_units, int half, int d,
                                 int n_future, double rope_base, float* __restrict__ coef) {
    int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= n_units * half) return;
    int u = t / half, m = t % half;
    double theta = exp2(-2.0 * (double)m / (double)d * log2(rope_base));
    double T = (double)n_future;
    double centre = ((double)pos_next[u] + 0.5 * (T - 1.0)) * theta;
    double sh = sin(0.5 * theta);
    // theta lies in (0, 1], so sin(theta/2) > 0; the guard only covers rope_base = inf.
    double ratio = (sh > 0.0) ? sin(0.5 * T * theta) / (T * sh) : 1.0;
    double sc, cc;
    sincos(centre, &sc, &cc);
    coef[2 * (size_t)t] = (float)(cc * ratio);
    coef[2 * (size_t)t + 1] = (float)(sc * ratio);
}

constexpr int kStatsThreads = 256;
constexpr int kRowBlock = 64;    // rows of Sigma_bar per CTA
constexpr int kWChunk = 32;      // window rows staged per step

template <int D>
__global__ void __launch_bounds__(kStatsThreads)
stats_kernel(const __nv_bfloat16* __restrict__ q_win, const float* __restrict__ coef, int Hq, int W,
             int layout, float inv_norm, float* __restrict__ mu_bar, float* __restrict__ sigma_bar) {
    constexpr int HALF = D / 2;
    constexpr int CT = D / 32;                     // columns per thread
    __shared__ float mu_s[D];
    __shared__ float c_s[HALF], s_s[HALF];
    __shared__ __align__(16) float x_s[kWChunk][D];

    const int uh = blockIdx.x;
    const int u = uh / Hq;
    const int rb = blockIdx.y;
    const int tid = threadIdx.x;
    const __nv_bfloat16* q = q_win + (size_t)uh * W * D;

    for (int m = tid; m < HALF; m += kStatsThreads) {
        c_s[m] = coef[2 * ((size_t)u * HALF + m)];
        s_s[m] = coef[2 * ((size_t)u * HALF + m) + 1];
    }
    for (int c = tid; c < D; c += kStatsThreads) {
        float acc = 0.f;
        for (int w = 0; w < W; ++w) acc += __bfloat162float(q[(size_t)w * D + c]);
        mu_s[c] = acc / (float)W;
    }
    __syncthreads();

    if (rb == 0) {
        for (int m = tid; m < HALF; m += kStatsThreads) {
            int a = layout == EA_ROPE_INTERLEAVED ? 2 * m : m;
            int b = layout == EA_ROPE_INTERLEAVED ? 2 * m + 1 : m + HALF;
            float ma = mu_s[a], mb = mu_s[b];
            mu_bar[(size_t)uh * D + a] = c_s[m] * ma - s_s[m] * mb;
            mu_bar[(size_t)uh * D + b] = s_s[m] * ma + c_s[m] * mb;
        }
    }

    const int ty = tid / 32, tx = tid % 32;
    const int row0 = rb * kRowBlock + ty * 8;
    float acc[8][CT];
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < CT; ++j) acc[i][j] = 0.f;

    for (int w0 = 0; w0 < W; w0 += kWChunk) {
        const int rows = min(kWChunk, W - w0);
        __syncthreads();
        // stage x_w = R_bar (u_w - mu) for this chunk of window rows
        for (int e = tid; e < kWChunk * HALF; e += kStatsThreads) {
            int w = e / HALF, m = e % HALF;
            int a = layout == EA_ROPE_INTERLEAVED ? 2 * m : m;
            int b = layout == EA_ROPE_INTERLEAVED ? 2 * m + 1 : m + HALF;
            float xa = 0.f, xb = 0.f;
            if (w < rows) {
                xa = __bfloat162float(q[(size_t)(w0 + w) * D + a]) - mu_s[a];
                xb = __bfloat162float(q[(size_t)(w0 + w) * D + b]) - mu_s[b];
            }
            x_s[w][a] = c_s[m] * xa - s_s[m] * xb;
            x_s[w][b] = s_s[m] * xa + c_s[m] * xb;
        }
        __syncthreads();
#pragma unroll 4
        for (int w = 0; w < kWChunk; ++w) {
            float r[8], c[CT];
            const float4 r0 = *reinterpret_cast<const float4*>(&x_s[w][row0]);
            const float4 r1 = *reinterpret_cast<const float4*>(&x_s[w][row0 + 4]);
            r[0] = r0.x; r[1] = r0.y; r[2] = r0.z; r[3] = r0.w;
            r[4] = r1.x; r[5] = r1.y; r[6] = r1.z; r[7] = r1.w;
#pragma unroll
            for (int j = 0; j < CT; ++j) c[j] = x_s[w][tx + 32 * j];
#pragma unroll
            for (int i = 0; i < 8; ++i)
#pragma unroll
                for (int j = 0; j < CT; ++j) acc[i][j] = fmaf(r[i], c[j], acc[i][j]);
        }
    }

    float* out = sigma_bar + (size_t)uh * D * D;
#pragma unroll
    for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < CT; ++j)
            out[(size_t)(row0 + i) * D + tx + 32 * j] = acc[i][j] * inv_norm;
}

}  // namespace

ea_status ea_launch_stats(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* q_win,
                          const int64_t* pos_next, int n_future, double rope_base, float* rope_coef,
                          float* mu_bar, float* sigma_bar, cudaStream_t st) {
    const int d = s.head_dim, half = d / 2;
    const int n_coef = s.n_units * half;
    rope_coef_kernel<<<(n_coef + 127) / 128, 128, 0, st>>>(pos_next, s.n_units, half, d, n_future,
                                                           rope_base, rope_coef);
    const float inv_norm =
        1.0f / (float)(s.cov_norm == EA_COV_SAMPLE ? s.window - 1 : s.window);
    dim3 grid((unsigned)(s.n_units * s.n_q_heads), (unsigned)(d / kRowBlock));
    switch (d) {
        case 64:
            stats_kernel<64><<<grid, kStatsThreads, 0, st>>>(q_win, rope_coef, s.n_q_heads, s.window,
                                                            s.rope_layout, inv_norm, mu_bar, sigma_bar);
            break;
        case 128:
            stats_kernel<128><<<grid, kStatsThreads, 0, st>>>(q_win, rope_coef, s.n_q_heads, s.window,
                                                             s.rope_layout, inv_norm, mu_bar, sigma_bar);
            break;
        case 256:
            stats_kernel<256><<<grid, kStatsThreads, 0, st>>>(q_win, rope_coef, s.n_q_heads, s.window,
                                                             s.rope_layout, inv_norm, mu_bar, sigma_bar);
            break;
        default:
            return EA_ERR_UNSUPPORTED;
    }
    ea_count_launches(ctx, 2);
    return cudaGetLastError() == cudaSuccess ? EA_OK : EA_ERR_CUDA;
}

// ---------------------------------------------------------------------------------------------
// ea_query_stats_static: the same two kernels, with the averaged-rotation coefficients kept in a
// fixed device array of this library instead of a context workspace.  Nothing is allocated here
// or on first use; the array is part of the loaded module on every GPU that loads the library.
#include <mutex>

namespace {

// fp32 (cos, sin) pairs: n_units * head_dim / 2 of them per call.
static __device__ __align__(256) float g_static_rope_coef[2 * EA_STATIC_MAX_ROPE_PAIRS];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
float* g_static_coef_addr[kMaxDevices];   // device address of the array, per device, once resolved

// Device address of g_static_rope_coef on the CURRENT device.  The symbol's name is only a
// host-side handle; kernels must be given the address the runtime reports for it.
ea_status static_coef_address(float** out) {
    int dev = 0;
    EA_CUDA_TRY(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return EA_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    if (!g_static_coef_addr[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_rope_coef) != cudaSuccess || !ptr) {
            cudaGetLastError();
            return EA_ERR_CUDA;
        }
        g_static_coef_addr[dev] = static_cast<float*>(ptr);
    }
    *out = g_static_coef_addr[dev];
    return EA_OK;
}

}  // namespace

extern "C" ea_status ea_query_stats_static(const ea_shape* s, const void* q_win, const int64_t* pos_next,
                                           int32_t n_future, double rope_base, float* mu_bar,
                                           float* sigma_bar, void* cuda_stream) {
    if (!s) return EA_ERR_INVALID_ARG;
    if (s->n_units < 0 || s->n_q_heads < 1 || s->window < 1) return EA_ERR_INVALID_ARG;
    if (s->rope_layout != EA_ROPE_HALF_SPLIT && s->rope_layout != EA_ROPE_INTERLEAVED) return EA_ERR_INVALID_ARG;
    if (s->cov_norm != EA_COV_POPULATION && s->cov_norm != EA_COV_SAMPLE) return EA_ERR_INVALID_ARG;
    if (s->cov_norm == EA_COV_SAMPLE && s->window < 2) return EA_ERR_INVALID_ARG;
    if (s->head_dim != 64 && s->head_dim != 128 && s->head_dim != 256) return EA_ERR_UNSUPPORTED;
    if (n_future < 1 || !(rope_base > 0.0)) return EA_ERR_INVALID_ARG;
    const int d = s->head_dim, half = d / 2;
    // the fixed array bounds the problem size: refuse anything that would not fit
    if ((long long)s->n_units * half > (long long)EA_STATIC_MAX_ROPE_PAIRS) return EA_ERR_WORKSPACE;
    if ((long long)s->n_units * s->n_q_heads > 0x7fffffffLL) return EA_ERR_UNSUPPORTED;
    if (s->n_units == 0) return EA_OK;
    if (!q_win || !pos_next || !mu_bar || !sigma_bar) return EA_ERR_INVALID_ARG;
    if (((uintptr_t)q_win | (uintptr_t)mu_bar | (uintptr_t)sigma_bar) & 15u) return EA_ERR_INVALID_ARG;

    float* coef = nullptr;
    ea_status st = static_coef_address(&coef);
    if (st != EA_OK) return st;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const __nv_bfloat16* q = static_cast<const __nv_bfloat16*>(q_win);
    const int n_coef = s->n_units * half;
    // every coefficient this call reads is written first, so stale contents of earlier calls are harmless
    rope_coef_kernel<<<(n_coef + 127) / 128, 128, 0, stream>>>(pos_next, s->n_units, half, d, n_future,
                                                               rope_base, coef);
    const float inv_norm = 1.0f / (float)(s->cov_norm == EA_COV_SAMPLE ? s->window - 1 : s->window);
    dim3 grid((unsigned)(s->n_units * s->n_q_heads), (unsigned)(d / kRowBlock));
    switch (d) {
        case 64:
            stats_kernel<64><<<grid, kStatsThreads, 0, stream>>>(q, coef, s->n_q_heads, s->window,
                                                                 s->rope_layout, inv_norm, mu_bar, sigma_bar);
            break;
        case 128:
            stats_kernel<128><<<grid, kStatsThreads, 0, stream>>>(q, coef, s->n_q_heads, s->window,
                                                                  s->rope_layout, inv_norm, mu_bar, sigma_bar);
            break;
        default:
            stats_kernel<256><<<grid, kStatsThreads, 0, stream>>>(q, coef, s->n_q_heads, s->window,
                                                                  s->rope_layout, inv_norm, mu_bar, sigma_bar);
            break;
    }
    return cudaGetLastError() == cudaSuccess ? EA_OK : EA_ERR_CUDA;
}
