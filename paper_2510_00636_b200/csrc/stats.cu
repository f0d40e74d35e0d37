// Query statistics with the rotary embedding averaged over future positions
// (Eq. 5 and Eq. 6 of the paper, window queries given directly).
//
// Kernel 1 (rope_coef_kernel): for each unit and rotation pair m, the mean of
// cos/sin(p * theta_m) over p = pos_next .. pos_next + T - 1, evaluated in fp64
// with the closed form of the geometric series
//   (1/T) sum_j e^{i theta (p+j)} = e^{i theta (p + (T-1)/2)} sin(T theta/2) / (T sin(theta/2)).
// Kernel 2 (stats_mma_kernel): per query head, mu_bar = R_bar mu and
//   Sigma_bar = (1/N) sum_w x_w x_w^T,  x_w = R_bar (u_w - mu),
// which equals R_bar Sigma R_bar^T.  Tensor cores on a bf16 (hi, lo) pair of x, fp32 accumulation.
#include "ea_internal.h"
#include "image_layout.cuh"

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

// ---------------------------------------------------------------------------------------------
// Sigma_bar = (1/N) X^T X with X[w] = R_bar (u_w - mu) is a
// symmetric rank-W update; each CTA computes one BM x BM block of the upper triangle with
// mma.sync.m16n8k16 (bf16 x bf16 -> fp32).  X is kept as a bf16 pair (hi, lo) and three products
// (hi.hi + hi.lo + lo.hi) are accumulated, so every product carries 16 significant bits of each
// factor; the lower triangle is a copy of the upper one, which makes the result bitwise symmetric.
// X is staged as it lies, [window row][channel]: both MMA operands want the window index as their
// contraction index, which ldmatrix.trans delivers from that layout, so nothing is transposed on the way.
constexpr int kKC = 32;            // window rows per shared-memory chunk

// four 8x8 bf16 matrices, each stored as 8 rows (contraction index) of 8 contiguous elements, transposed
// into the fragment layout of mma.m16n8k16
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
// two such matrices (lanes 0-15 give the row addresses)
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t addr, uint32_t (&r)[2]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];"
                 : "=r"(r[0]), "=r"(r[1])
                 : "r"(addr));
}
// eight consecutive channels of a window row
__device__ __forceinline__ void load8(const __nv_bfloat16* p, float (&v)[8]) {
    const uint4 x = __ldg(reinterpret_cast<const uint4*>(p));
    const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}
__device__ __forceinline__ void load8(const float* p, float (&v)[8]) {
    const float4 a = __ldg(reinterpret_cast<const float4*>(p)), b = __ldg(reinterpret_cast<const float4*>(p) + 1);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}
__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Fused mode (ea_set_fused_stats): the statistics kernel also writes, from its accumulators, the bf16
// covariance image that the log-score kernel loads (what sigma_image_kernel would build from sigma_bar),
// so that ea_score needs neither that kernel nor sigma_bar.  image == nullptr: off.
struct StatsImage {
    uint8_t* image;      // images of the call, one per (unit, KV head, head subset)
    float* vec;          // fp32 [units * Hq, d] diagonals
    int Hkv;
    float lin_scale;     // 1 / sqrt(d)
    float quad_scale;    // 1 / (2 d)
};

// Shared memory: the staged chunk (hi and lo, kKC rows of the block's channels, padded by 16 bytes so that
// the eight rows of an 8x8 matrix fall into different banks), which the fused image's tile reuses; then
// the mean, the averaged rotation and the partial sums of the mean.
template <int D>
struct StatsGeo {
    static constexpr int BM = D < 128 ? D : 128;          // block edge
    static constexpr int NB1 = D / BM;                    // blocks per edge (1 or 2)
    static constexpr int PITCH = (NB1 == 1 ? BM : 2 * BM) + 8;       // bf16 per staged window row
    static constexpr int STAGE = 2 * kKC * PITCH * 2;
    static constexpr int TILE = NB1 == 1 ? EaImage<D>::KCH * D * 128 : 0;
    static constexpr int REGION = STAGE > TILE ? STAGE : TILE;
    static constexpr int SMEM = REGION + (D + D) * 4 + (256 / (D / 2)) * D * 4;
};

// packed fp32 pair arithmetic (two lanes per instruction)
__device__ __forceinline__ float2 fma2(float2 a, float2 b, float2 c) {
    float2 d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;"
        : "=l"(reinterpret_cast<uint64_t&>(d))
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)), "l"(reinterpret_cast<uint64_t&>(c)));
    return d;
}
__device__ __forceinline__ float2 mul2(float2 a, float2 b) {
    float2 d;
    asm("mul.rn.f32x2 %0, %1, %2;"
        : "=l"(reinterpret_cast<uint64_t&>(d))
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)));
    return d;
}
__device__ __forceinline__ float2 sub2(float2 a, float2 b) {
    float2 d;
    asm("sub.rn.f32x2 %0, %1, %2;"
        : "=l"(reinterpret_cast<uint64_t&>(d))
        : "l"(reinterpret_cast<uint64_t&>(a)), "l"(reinterpret_cast<uint64_t&>(b)));
    return d;
}
// eight consecutive floats from shared memory, 16-byte aligned
__device__ __forceinline__ void lds8(const float* p, float (&v)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p), b = *reinterpret_cast<const float4*>(p + 4);
    v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w;
    v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
}

// Where the accumulator tiles (16 channel rows x 8 channel columns, one mma.m16n8k16 each) of a warp lie in
// the CTA's BM x BM block.
//   full block (TRI = false): the warps form a 2 x 4 grid of (BM/2) x (BM/4) warp tiles.
//   upper triangle of a diagonal block of 128 (TRI = true): the block has 8 strips of 16 rows; strip i needs
//   the column tiles j >= 2 i (the two that straddle the diagonal included): 72 of the 128 tiles, nine per
//   warp.  Warp 2p takes strip p, columns 2p .. 2p+8; warp 2p+1 the rest of strip p (columns 2p+9 .. 15)
//   and all of strip 7-p (columns 14-2p .. 15).  A warp's tile 0 is the single odd column tile, tiles 1 .. 8
//   are four pairs of neighbouring column tiles, so that one ldmatrix.x4 serves a pair.
template <int BM, bool TRI>
struct StatsTiles {
    static constexpr int TM = BM / 32, TN = BM / 32;      // full block: mma tiles per warp along rows, columns
    static constexpr int NT = TRI ? 9 : TM * TN;
    int p, q;                                             // TRI: warp = 2p + q
    int wm, wn;                                           // full: warp position
    __device__ __forceinline__ explicit StatsTiles(int warp) : p(warp / 2), q(warp % 2), wm(warp / 4), wn(warp % 4) {}
    // TRI: the strip (0: strip p, 1: strip 7-p) and first column tile of pair r
    __device__ __forceinline__ int pair_second_strip(int r) const { return q && r >= 3 - p; }
    __device__ __forceinline__ int pair_col(int r) const {
        if (!q) return 2 * p + 2 * r;
        return r < 3 - p ? 2 * p + 10 + 2 * r : 14 - 2 * p + 2 * (r - (3 - p));
    }
    __device__ __forceinline__ int row0(int t) const {    // first channel row of tile t within the block
        if (!TRI) return wm * (BM / 2) + (t / TN) * 16;
        return 16 * ((t > 0 && pair_second_strip((t - 1) / 2)) ? 7 - p : p);
    }
    __device__ __forceinline__ int col0(int t) const {    // first channel column of tile t within the block
        if (!TRI) return wn * (BM / 4) + (t % TN) * 8;
        if (t == 0) return 8 * (q ? 2 * p + 9 : 2 * p + 8);
        return 8 * (pair_col((t - 1) / 2) + (t - 1) % 2);
    }
};

// QT: the window queries as bf16 (what a model's query projection emits) or fp32 (from project_kernel).
// TRI: the CTA computes the upper triangle of diagonal block blockIdx.y (blocks of 128 only); otherwise the
// whole block (0, 0) (head_dim 64) or (0, 1) (head_dim 256).
template <int D, typename QT, bool TRI>
__global__ void __launch_bounds__(256, TRI ? 3 : 2)
stats_mma_kernel(const QT* __restrict__ q_win, const float* __restrict__ coef, int Hq, int W,
                 int layout, float inv_norm, float* __restrict__ mu_bar, float* __restrict__ sigma_bar,
                 int w_cap, const long long* __restrict__ pushed, int cov_sample, const StatsImage img) {
    using SG = StatsGeo<D>;
    constexpr int HALF = D / 2;
    constexpr int BM = SG::BM, NB1 = SG::NB1, P = SG::PITCH;
    using TL = StatsTiles<BM, TRI>;
    constexpr int WM = BM / 2, WN = BM / 4;        // full block: warp tile of the 2 x 4 warps
    constexpr int TM = TL::TM, TN = TL::TN, NT = TL::NT;
    static_assert(!TRI || BM == 128, "the triangular tiling is laid out for blocks of 128");
    extern __shared__ __align__(16) unsigned char stats_smem[];
    // [hi / lo][w in chunk][channel: BM channels of the block's rows, then (off the diagonal) of its columns]
    float* mu_s = reinterpret_cast<float*>(stats_smem + SG::REGION);                        // [D]
    float* c_s = mu_s + D;                                                                  // [HALF]
    float* s_s = c_s + HALF;                                                                // [HALF]
    float* red = s_s + HALF;                                                                // [256 / (D/2)][D]

    const int uh = blockIdx.x;
    const int u = uh / Hq;
    // the block (bi <= bj) of this CTA
    const int bi = TRI ? (int)blockIdx.y : 0;
    const int bj = TRI ? (int)blockIdx.y : NB1 - 1;
    const bool diag = bi == bj;
    const bool first_block = (TRI || NB1 == 1) && blockIdx.y == 0;      // writes mu_bar
    const int tid = threadIdx.x, lane = tid % 32, warp = tid / 32;
    // A window kept as a ring of w_cap rows (pushed != nullptr): the rows written so far, at most
    // w_cap of them, are the window; mean and covariance do not depend on their order, so a
    // wrapped ring is read as it lies and a partly filled one by its first rows.
    if (pushed) {
        const long long p = pushed[u];
        W = p < (long long)w_cap ? (int)p : w_cap;
        // nothing to estimate from: zero statistics (uniform expected attention); the loops below then run
        // over no rows and every output is written as zero
        if (W < 1 + cov_sample) { W = 0; inv_norm = 0.f; }
        else         inv_norm = 1.0f / (float)(W - cov_sample);
    }
    const QT* q = q_win + (size_t)uh * w_cap * D;

    for (int m = tid; m < HALF; m += 256) {
        c_s[m] = coef[2 * ((size_t)u * HALF + m)];
        s_s[m] = coef[2 * ((size_t)u * HALF + m) + 1];
    }
    {   // mean: thread = (group of window rows, channel pair); groups meet in shared memory
        constexpr int NG = 256 / HALF;
        const int cp = tid % HALF, g = tid / HALF;
        float a0 = 0.f, a1 = 0.f;
        if constexpr (sizeof(QT) == 2) {
            const uint32_t* q2 = reinterpret_cast<const uint32_t*>(q);
#pragma unroll 4
            for (int w = g; w < W; w += NG) {
                const uint32_t x = __ldg(q2 + (size_t)w * HALF + cp);
                a0 += __uint_as_float(x << 16);
                a1 += __uint_as_float(x & 0xffff0000u);
            }
        } else {
            const float2* q2 = reinterpret_cast<const float2*>(q);
#pragma unroll 4
            for (int w = g; w < W; w += NG) {
                const float2 x = __ldg(q2 + (size_t)w * HALF + cp);
                a0 += x.x;
                a1 += x.y;
            }
        }
        red[g * D + 2 * cp] = a0;
        red[g * D + 2 * cp + 1] = a1;
        __syncthreads();
        for (int c = tid; c < D; c += 256) {
            float acc = 0.f;
#pragma unroll
            for (int gg = 0; gg < NG; ++gg) acc += red[gg * D + c];      // fixed order
            mu_s[c] = W > 0 ? acc / (float)W : 0.f;
        }
    }
    __syncthreads();
    if (first_block) {
        for (int m = tid; m < HALF; m += 256) {
            const int a = layout == EA_ROPE_INTERLEAVED ? 2 * m : m;
            const int b = layout == EA_ROPE_INTERLEAVED ? 2 * m + 1 : m + HALF;
            const float ma = mu_s[a], mb = mu_s[b];
            const float ra = c_s[m] * ma - s_s[m] * mb, rb = s_s[m] * ma + c_s[m] * mb;
            mu_bar[(size_t)uh * D + a] = ra;
            mu_bar[(size_t)uh * D + b] = rb;
            red[a] = ra;                       // (the mean's partial sums are no longer needed) for the fused image
            red[b] = rb;
        }
    }

    float acc[NT][4];
#pragma unroll
    for (int t = 0; t < NT; ++t)
#pragma unroll
        for (int e = 0; e < 4; ++e) acc[t][e] = 0.f;

    const TL tiles(warp);
    const int wm = tiles.wm, wn = tiles.wn;
    const int n_ch = diag ? BM : 2 * BM;           // channels staged per chunk
    const uint32_t xs_hi = static_cast<uint32_t>(__cvta_generic_to_shared(stats_smem));
    const uint32_t xs_lo = xs_hi + kKC * P * 2;

    // This thread's eight staged channels (one 16-byte piece of a row; the same for the whole kernel), the
    // channels they rotate with, and where the averaged rotation's coefficients of the pairs start:
    //   x[ch] = c_m (u_ch - mu_ch) -/+ s_m (u_partner - mu_partner),  minus for the first channel of a pair.
    const int pieces = n_ch / 8, t_p = tid % pieces, t_w = tid / pieces, t_wstep = 256 / pieces;
    const int sc0 = 8 * t_p;
    const int ch0 = (sc0 < BM ? bi * BM : bj * BM - BM) + sc0;
    const bool interleaved = layout == EA_ROPE_INTERLEAVED;
    const bool first_side = ch0 < HALF;                      // (half-split layout) the piece holds first channels
    const int pch0 = interleaved ? ch0 : (first_side ? ch0 + HALF : ch0 - HALF);
    const int m0 = interleaved ? ch0 / 2 : (first_side ? ch0 : ch0 - HALF);

    for (int w0 = 0; w0 < W; w0 += kKC) {
        __syncthreads();
        for (int w = t_w; w < kKC; w += t_wstep) {
            uint32_t hi[4] = {0u, 0u, 0u, 0u}, lo[4] = {0u, 0u, 0u, 0u};
            if (w0 + w < W) {
                float uo[8], up[8];
                load8(q + (size_t)(w0 + w) * D + ch0, uo);
                if (interleaved) {
#pragma unroll
                    for (int i = 0; i < 8; ++i) up[i] = uo[i ^ 1];
                } else {
                    load8(q + (size_t)(w0 + w) * D + pch0, up);
                }
                float mo[8], mp[8], cm[8], sm[8];
                lds8(mu_s + ch0, mo);
                // (interleaved pairs: four coefficient pairs serve the piece; the second half of these loads is
                // not used and may run four entries into the array that follows in shared memory)
                lds8(mu_s + pch0, mp);
                lds8(c_s + m0, cm);
                lds8(s_s + m0, sm);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    // two channels at a time with packed fp32 arithmetic and packed conversions
                    float2 tc, ts, mpp;
                    if (interleaved) {
                        tc = make_float2(cm[i], cm[i]);
                        ts = make_float2(-sm[i], sm[i]);
                        mpp = make_float2(mp[2 * i + 1], mp[2 * i]);
                    } else {
                        tc = make_float2(cm[2 * i], cm[2 * i + 1]);
                        ts = first_side ? make_float2(-sm[2 * i], -sm[2 * i + 1]) : make_float2(sm[2 * i], sm[2 * i + 1]);
                        mpp = make_float2(mp[2 * i], mp[2 * i + 1]);
                    }
                    const float2 xa = sub2(make_float2(uo[2 * i], uo[2 * i + 1]), make_float2(mo[2 * i], mo[2 * i + 1]));
                    const float2 xb = sub2(make_float2(up[2 * i], up[2 * i + 1]), mpp);
                    const float2 x = fma2(tc, xa, mul2(ts, xb));
                    const __nv_bfloat162 h = __floats2bfloat162_rn(x.x, x.y);
                    const uint32_t hb = *reinterpret_cast<const uint32_t*>(&h);
                    const float2 r = sub2(x, make_float2(__uint_as_float(hb << 16), __uint_as_float(hb & 0xffff0000u)));
                    const __nv_bfloat162 l = __floats2bfloat162_rn(r.x, r.y);
                    hi[i] = hb;
                    lo[i] = *reinterpret_cast<const uint32_t*>(&l);
                }
            }
            // rows past the window are zero
            *reinterpret_cast<uint4*>(stats_smem + (w * P + sc0) * 2) = make_uint4(hi[0], hi[1], hi[2], hi[3]);
            *reinterpret_cast<uint4*>(stats_smem + ((kKC + w) * P + sc0) * 2) = make_uint4(lo[0], lo[1], lo[2], lo[3]);
        }
        __syncthreads();
#pragma unroll
        for (int k0 = 0; k0 < kKC; k0 += 16) {
            if constexpr (TRI) {
                // A fragments of the warp's one or two strips; matrices (channels +0, w +0), (+8, +0), (+0, +8), (+8, +8)
                uint32_t a_hi[2][4], a_lo[2][4];
                const int kr_a = k0 + (lane % 8) + 8 * (lane / 16);
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int mc = 16 * (i ? (tiles.q ? 7 - tiles.p : tiles.p) : tiles.p) + 8 * ((lane / 8) % 2);
                    const uint32_t off = (uint32_t)((kr_a * P + mc) * 2);
                    ldmatrix_x4_trans(xs_hi + off, a_hi[i]);
                    ldmatrix_x4_trans(xs_lo + off, a_lo[i]);
                }
                {   // tile 0: the single column tile, always in strip p; matrices (w +0), (w +8)
                    uint32_t b_hi[2], b_lo[2];
                    const int kr = k0 + (lane % 8) + 8 * ((lane / 8) % 2);
                    const uint32_t off = (uint32_t)((kr * P + tiles.col0(0)) * 2);
                    ldmatrix_x2_trans(xs_hi + off, b_hi);
                    ldmatrix_x2_trans(xs_lo + off, b_lo);
                    mma_bf16_16816(acc[0], a_hi[0], b_hi[0], b_hi[1]);
                    mma_bf16_16816(acc[0], a_hi[0], b_lo[0], b_lo[1]);
                    mma_bf16_16816(acc[0], a_lo[0], b_hi[0], b_hi[1]);
                }
#pragma unroll
                for (int r = 0; r < 4; ++r) {
                    // a pair of column tiles: (tile 0, w +0), (tile 0, w +8), (tile 1, w +0), (tile 1, w +8)
                    uint32_t b_hi[4], b_lo[4];
                    const int kr = k0 + (lane % 8) + 8 * ((lane / 8) % 2);
                    const int nc = 8 * tiles.pair_col(r) + 8 * (lane / 16);
                    const uint32_t off = (uint32_t)((kr * P + nc) * 2);
                    ldmatrix_x4_trans(xs_hi + off, b_hi);
                    ldmatrix_x4_trans(xs_lo + off, b_lo);
                    if (tiles.pair_second_strip(r)) {          // warp-uniform
#pragma unroll
                        for (int jj = 0; jj < 2; ++jj) {
                            mma_bf16_16816(acc[1 + 2 * r + jj], a_hi[1], b_hi[2 * jj], b_hi[2 * jj + 1]);
                            mma_bf16_16816(acc[1 + 2 * r + jj], a_hi[1], b_lo[2 * jj], b_lo[2 * jj + 1]);
                            mma_bf16_16816(acc[1 + 2 * r + jj], a_lo[1], b_hi[2 * jj], b_hi[2 * jj + 1]);
                        }
                    } else {
#pragma unroll
                        for (int jj = 0; jj < 2; ++jj) {
                            mma_bf16_16816(acc[1 + 2 * r + jj], a_hi[0], b_hi[2 * jj], b_hi[2 * jj + 1]);
                            mma_bf16_16816(acc[1 + 2 * r + jj], a_hi[0], b_lo[2 * jj], b_lo[2 * jj + 1]);
                            mma_bf16_16816(acc[1 + 2 * r + jj], a_lo[0], b_hi[2 * jj], b_hi[2 * jj + 1]);
                        }
                    }
                }
            } else {
                uint32_t a_hi[TM][4], a_lo[TM][4];
#pragma unroll
                for (int i = 0; i < TM; ++i) {
                    // matrices: (channels +0, w +0), (channels +8, w +0), (channels +0, w +8), (channels +8, w +8)
                    const int kr = k0 + (lane % 8) + 8 * (lane / 16);
                    const int mc = wm * WM + i * 16 + 8 * ((lane / 8) % 2);
                    const uint32_t off = (uint32_t)((kr * P + mc) * 2);
                    ldmatrix_x4_trans(xs_hi + off, a_hi[i]);
                    ldmatrix_x4_trans(xs_lo + off, a_lo[i]);
                }
#pragma unroll
                for (int j2 = 0; j2 < TN; j2 += 2) {
                    // two 8-channel column tiles per load: (tile 0, w +0), (tile 0, w +8), (tile 1, w +0), (tile 1, w +8)
                    uint32_t b_hi[4], b_lo[4];
                    const int kr = k0 + (lane % 8) + 8 * ((lane / 8) % 2);
                    const int nc = (diag ? 0 : BM) + wn * WN + j2 * 8 + 8 * (lane / 16);
                    const uint32_t off = (uint32_t)((kr * P + nc) * 2);
                    ldmatrix_x4_trans(xs_hi + off, b_hi);
                    ldmatrix_x4_trans(xs_lo + off, b_lo);
#pragma unroll
                    for (int i = 0; i < TM; ++i)
#pragma unroll
                        for (int jj = 0; jj < 2; ++jj) {
                            mma_bf16_16816(acc[i * TN + j2 + jj], a_hi[i], b_hi[2 * jj], b_hi[2 * jj + 1]);
                            mma_bf16_16816(acc[i * TN + j2 + jj], a_hi[i], b_lo[2 * jj], b_lo[2 * jj + 1]);
                            mma_bf16_16816(acc[i * TN + j2 + jj], a_lo[i], b_hi[2 * jj], b_hi[2 * jj + 1]);
                        }
                }
            }
        }
    }

    // upper triangle from the accumulators, lower triangle as its mirror
    if (sigma_bar) {
        float* out = sigma_bar + (size_t)uh * D * D;
#pragma unroll
        for (int t = 0; t < NT; ++t)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int a = bi * BM + tiles.row0(t) + lane / 4 + 8 * (e / 2);
                const int c = bj * BM + tiles.col0(t) + 2 * (lane % 4) + (e % 2);
                if (a <= c) {
                    const float v = acc[t][e] * inv_norm;
                    out[(size_t)a * D + c] = v;
                    out[(size_t)c * D + a] = v;
                }
            }
    }
    if constexpr (NB1 == 1) {
        if (img.image) {
            // ---- the covariance image of this head, bit for bit what sigma_image_kernel builds from sigma_bar
            using L = EaImage<D>;
            const int h = uh % Hq, Gq = Hq / img.Hkv;
            const int g = h / Gq, hg = h % Gq;
            const int n_subsets = (Gq + L::HPC - 1) / L::HPC;
            const int hs = hg / L::HPC, jh = hg % L::HPC;
            uint8_t* gimg = img.image + ((size_t)(u * img.Hkv + g) * n_subsets + hs) * L::IMG_FULL;
            __syncthreads();                              // the staging buffers of the main loop are dead
            // tile[kc][c][128 bytes]: this head's rows in channel order, swizzled as in the image (the image
            // row of channel c has the same low three bits as c)
            uint8_t* tile = stats_smem;
            float* dg_s = red + D;                         // [D] diagonal of Sigma_bar / (2 d)
            auto at = [&](int r, int k) {
                return reinterpret_cast<__nv_bfloat16*>(tile + (k / 64) * (D * 128) + r * 128 +
                                                        ((((k % 64) / 8) ^ (r & 7)) << 4) + (k % 8) * 2);
            };
#pragma unroll
            for (int t = 0; t < NT; ++t)
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        const int a = tiles.row0(t) + lane / 4 + 8 * (e / 2);
                        const int c = tiles.col0(t) + 2 * (lane % 4) + (e % 2);
                        const float v = acc[t][e] * inv_norm;
                        if (a < c) {
                            // the two mirrored entries together carry (S_ca + S_ac) / (2 d), split into a bf16
                            // and the bf16 rounding of its remainder
                            const float x = (v + v) * img.quad_scale;
                            const __nv_bfloat16 hi = __float2bfloat16_rn(x);
                            *at(c, a) = hi;
                            *at(a, c) = __float2bfloat16_rn(x - __bfloat162float(hi));
                        } else if (a == c) {
                            const float dg = v * img.quad_scale;
                            *at(c, c) = __float2bfloat16_rn(dg);     // its bf16 part; the rest in the diagonal blocks
                            dg_s[c] = dg;
                        }
                    }
            __syncthreads();
            for (int e = tid; e < L::KCH * D * 8; e += 256) {
                const int piece = e % 8, c = (e / 8) % D, kc = e / (8 * D);
                const uint4 x = *reinterpret_cast<const uint4*>(tile + kc * (D * 128) + c * 128 + piece * 16);
                *reinterpret_cast<uint4*>(gimg + (size_t)kc * L::CHUNK_B_FULL + (size_t)L::col(jh, c) * 128 + piece * 16) = x;
            }
            // linear-term operand, diagonal vector and diagonal blocks (as sigma_image_kernel writes them)
            for (int c = tid; c < D; c += 256) {
                const float m = red[c] * img.lin_scale;
                const __nv_bfloat16 hi = __float2bfloat16_rn(m);
                const __nv_bfloat16 lo = __float2bfloat16_rn(m - __bfloat162float(hi));
                const int row = L::col(jh, c);
                uint8_t* dst = gimg + L::IMG_MAIN + (size_t)(row / 8) * 256 + (row % 8) * 16;
                *reinterpret_cast<uint4*>(dst) =
                    make_uint4((uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16), 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(dst + 128) = make_uint4(0u, 0u, 0u, 0u);
                const float dg = dg_s[c];
                img.vec[(size_t)uh * D + c] = dg;
                const __nv_bfloat16 dlo = __float2bfloat16_rn(dg - __bfloat162float(__float2bfloat16_rn(dg)));
                const int kk = c % 16, n = 16 * jh + kk;
                uint8_t* blk = gimg + L::IMG_MAIN + L::LIN_FULL + (size_t)(c / 16) * L::DIAG_BLOCK + (n / 8) * 256 + (n % 8) * 16;
                uint32_t w4[4] = {0u, 0u, 0u, 0u};
                w4[(kk % 8) / 2] = (uint32_t)__bfloat16_as_ushort(dlo) << (16 * (kk % 2));
                const uint4 mine = make_uint4(w4[0], w4[1], w4[2], w4[3]), zero = make_uint4(0u, 0u, 0u, 0u);
                *reinterpret_cast<uint4*>(blk) = kk < 8 ? mine : zero;
                *reinterpret_cast<uint4*>(blk + 128) = kk < 8 ? zero : mine;
            }
        }
    }
}

}  // namespace

template <typename QT>
static ea_status launch_stats(const ea_ctx* ctx, const ea_shape& s, const QT* q_win, const int64_t* pos_next,
                              int n_future, double rope_base, float* rope_coef, float* mu_bar, float* sigma_bar,
                              cudaStream_t st, const int64_t* pushed = nullptr, void* image = nullptr,
                              float* vec = nullptr) {
    const int d = s.head_dim, half = d / 2;
    const int n_coef = s.n_units * half;
    rope_coef_kernel<<<(n_coef + 127) / 128, 128, 0, st>>>(pos_next, s.n_units, half, d, n_future,
                                                           rope_base, rope_coef);
    const float inv_norm =
        1.0f / (float)(s.cov_norm == EA_COV_SAMPLE ? s.window - 1 : s.window);
    const unsigned heads = (unsigned)(s.n_units * s.n_q_heads);
    const StatsImage img = {static_cast<uint8_t*>(image), vec, s.n_kv_heads, 1.0f / sqrtf((float)d), 0.5f / (float)d};
    int n_launches = 2;
    auto launch = [&](auto kern, int smem, unsigned blocks_y) {
        if (smem > 48 * 1024 &&
            cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem) != cudaSuccess)
            return false;
        kern<<<dim3(heads, blocks_y), 256, smem, st>>>(q_win, rope_coef, s.n_q_heads, s.window, s.rope_layout,
                                                       inv_norm, mu_bar, sigma_bar, s.window,
                                                       reinterpret_cast<const long long*>(pushed),
                                                       s.cov_norm == EA_COV_SAMPLE ? 1 : 0, img);
        return true;
    };
    bool ok;
    switch (d) {
        case 64: ok = launch(stats_mma_kernel<64, QT, false>, StatsGeo<64>::SMEM, 1); break;
        case 128: ok = launch(stats_mma_kernel<128, QT, true>, StatsGeo<128>::SMEM, 1); break;
        case 256:
            // the two diagonal blocks (upper triangles), then the block above the diagonal
            ok = launch(stats_mma_kernel<256, QT, true>, StatsGeo<256>::SMEM, 2) &&
                 launch(stats_mma_kernel<256, QT, false>, StatsGeo<256>::SMEM, 1);
            n_launches = 3;
            break;
        default: return EA_ERR_UNSUPPORTED;
    }
    if (!ok) return EA_ERR_CUDA;
    if (ctx) ea_count_launches(ctx, n_launches);
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_stats(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* q_win,
                          const int64_t* pos_next, int n_future, double rope_base, float* rope_coef,
                          float* mu_bar, float* sigma_bar, cudaStream_t st, void* image, float* vec) {
    return launch_stats(ctx, s, q_win, pos_next, n_future, rope_base, rope_coef, mu_bar, sigma_bar, st, nullptr, image,
                        vec);
}

ea_status ea_launch_stats_ring(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* q_ring,
                               const int64_t* pushed, const int64_t* pos_next, int n_future, double rope_base,
                               float* rope_coef, float* mu_bar, float* sigma_bar, cudaStream_t st, void* image,
                               float* vec) {
    return launch_stats(ctx, s, q_ring, pos_next, n_future, rope_base, rope_coef, mu_bar, sigma_bar, st, pushed, image,
                        vec);
}

ea_status ea_launch_stats_f32(const ea_ctx* ctx, const ea_shape& s, const float* q_win, const int64_t* pos_next,
                              int n_future, double rope_base, float* rope_coef, float* mu_bar, float* sigma_bar,
                              cudaStream_t st) {
    return launch_stats(ctx, s, q_win, pos_next, n_future, rope_base, rope_coef, mu_bar, sigma_bar, st);
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

    // the same launches as ea_query_stats, without a context (nothing to count the launches in); every
    // coefficient this call reads is written first, so stale contents of earlier calls are harmless
    return launch_stats(nullptr, *s, static_cast<const __nv_bfloat16*>(q_win), pos_next, n_future, rope_base, coef,
                        mu_bar, sigma_bar, static_cast<cudaStream_t>(cuda_stream));
}
