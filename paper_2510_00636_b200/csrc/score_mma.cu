// Log-scores s_{h,i} = mu_bar_h.k_i/sqrt(d) + k_i^T Sigma_bar_h k_i/(2d) (Eq. 7) on the
// tcgen05 tensor cores.
//
// The dense part is the product K . B^T of a tile of 128 cached keys with a bf16 image B of
// the covariance; the row-wise quadratic form is finished in the epilogue:
//     D[i, c]  = sum_a K[i, a] B[c, a]                      (tcgen05.mma, fp32 in tensor memory)
//                + mu_bar_c / sqrt(d)                        (one more MMA step: ones x (hi, lo) of the term)
//     s_{h,i}  = sum_c k_{i,c} ( D[i, c] + Sigma_bar_cc k_{i,c}/(2d) )
// B carries the off-diagonal of Sigma_bar/(2d) at twice bf16 precision for the price of one bf16
// matrix: the quadratic form only sees B[c,a] + B[a,c], so for a < c the entry B[c,a] holds
// bf16(Sigma_ac/d) and the mirrored entry B[a,c] holds the bf16 rounding of what that left over.
// At head_dim 256, where the tensor pipe is the limit, the diagonal stays out of B and enters in fp32
// in the epilogue (two FMAs per accumulator element).  At head_dim <= 128, where the epilogue is the
// limit, the diagonal goes through the tensor cores too, as a bf16 pair: its bf16 part on B's diagonal,
// the bf16 rounding of the rest by one small MMA (N = 16 heads-per-pass columns, K = 16) per 16
// channels against a diagonal block; the heads' accumulator columns are interleaved in runs of 16 so
// that one such step serves every head.  The epilogue is then s = sum_c k_c D[i, c]: one FMA per element.
//
// A CTA keeps the image of `hpc` query heads of one KV head resident in shared memory
// (hpc * d = 256 accumulator columns at most) and streams key tiles through a TMA ring:
//   warp 0     TMA producer (one lane): covariance image (bulk copy) and key tiles (tiled, 128B swizzle)
//   warp 1     MMA issuer (one lane); owns the tensor-memory allocation
//   warps 2-9  epilogue, two warps per tensor-memory lane quarter: thread <-> accumulator lane <-> key;
//              each reads its half of the key row and the matching accumulator columns, the halves of a
//              key meet in shared memory
// Tensor memory holds two accumulator stages so the epilogue of one tile overlaps the MMAs of the
// next.  With PAIR, two CTAs of a cluster work as one (cta_group::2): each stages its own 128 keys
// and half of the image rows, the leader issues M = 256 MMAs for both, and each CTA runs the
// epilogue of its own keys; this is what lets head_dim 256 fit in shared memory.
// Key tiles live in a ring of 16 KiB chunk slots (64 channels of 128 keys): two tiles deep at
// head_dim 256, four at head_dim <= 128.  The epilogue reads the key rows from the slots as it works
// through the accumulator and hands each slot back as soon as its warps are done with it.
// Every wait is bounded; a wait that gives up raises the context's status word.
#include <cuda_fp16.h>
#include <cuda_fp8.h>

#include <mutex>

#include "ea_internal.h"
#include "image_layout.cuh"
#include "ptx_sm100.cuh"

namespace {

using namespace ptx;

constexpr int kTileKeys = 128;                     // keys per CTA per step
constexpr int kTmemCols = 512;
constexpr int kAccCols = 256;                      // columns of one accumulator stage
constexpr int kChunkA = kTileKeys * 128;           // bytes of one 64-channel chunk of a key tile
constexpr int kChunkQ = kTileKeys * 64;            // the same chunk as FP8 codes

// Q8: the keys arrive as FP8 E4M3 codes.  The copy engine lands a chunk of codes (8 KiB) in the upper half
// of the chunk's 16 KiB slot of the operand ring; four more warps read them all, meet at a named barrier and
// write the bf16 values (exact) over the whole slot in the swizzled layout the MMA reads.  Everything
// downstream is unchanged.  Each CTA of a pair widens its own keys and reports them on the leader's barrier.
template <int D, bool PAIR, bool Q8 = false>
struct Geo {
    using L = EaImage<D>;                                // the image's layout in global memory
    static constexpr int HPC = L::HPC;
    static constexpr int KCH = L::KCH;
    static constexpr int IMG_ROWS = L::IMG_ROWS;
    static constexpr int CHUNK_B_FULL = L::CHUNK_B_FULL;
    static constexpr int IMG_MAIN = L::IMG_MAIN;
    static constexpr int ROWS_CTA = PAIR ? IMG_ROWS / 2 : IMG_ROWS;   // image rows one CTA keeps
    static constexpr int CHUNK_B = ROWS_CTA * 128;
    static constexpr int IMG_CTA = KCH * CHUNK_B;
    // Epilogue: EPI_PARTS warps per tensor-memory lane quarter, each with CPP columns of every head.
    static constexpr int EPI_PARTS = 2;
    static constexpr int EPI_WARPS = 4 * EPI_PARTS;
    static constexpr int CONV_WARPS = Q8 ? 4 : 0;          // warps 2 + EPI_WARPS ..: code -> bf16
    static constexpr int THREADS = 32 * (2 + EPI_WARPS + CONV_WARPS);
    static constexpr int CPP = D / EPI_PARTS;
    static constexpr int NSLOT = (D == 256 ? 2 : 4) * KCH;   // ring of 16 KiB chunk slots: 2 or 4 key tiles
    static constexpr int NQ = Q8 ? NSLOT : 0;              // "codes have landed" barriers, one per slot
    // arrivals that complete a ring slot: the copy engine's, or every widening warp's (of both CTAs of a pair)
    static constexpr int FILLERS = Q8 ? (PAIR ? 2 : 1) * CONV_WARPS : 1;
    static constexpr int VEC = HPC * D * (int)sizeof(float);       // diagonal vectors of the resident heads
    // linear term: one extra K = 16 MMA step, a constant block of ones times (hi, lo) of mu' per column,
    // both as unswizzled K-major core matrices (8 rows x 16 bytes; 128 bytes on along K, 256 on along rows)
    static constexpr int ONES = kTileKeys * 32;
    static constexpr int LIN_FULL = L::LIN_FULL;
    static constexpr int LIN_CTA = ROWS_CTA * 32;
    static constexpr bool DIAG_MMA = L::DIAG_MMA;
    static constexpr int DIAG_BLOCK = L::DIAG_BLOCK;
    static constexpr int DIAG_FULL = L::DIAG_FULL;
    __host__ __device__ static constexpr int col(int j, int c) { return L::col(j, c); }
    static constexpr int IMG_FULL = L::IMG_FULL;
    // partial sums of the column parts: [tile parity][part][head][key]
    static constexpr int PART = 2 * EPI_PARTS * HPC * kTileKeys * (int)sizeof(float);
    static constexpr int RED = HPC * 4 * 2 * (int)sizeof(float);   // per-warp (max, sum) of a work unit
    static constexpr int NBAR = 2 * NSLOT + 6 + NQ;
    static constexpr int CTRL = ((NBAR * 8 + 16) + 127) / 128 * 128;
    static constexpr int SMEM = IMG_CTA + NSLOT * kChunkA + ONES + LIN_CTA + VEC + DIAG_FULL + PART + RED + CTRL + 1024;
    // epilogue warps that read a chunk slot and hand it back to the producer
    static constexpr int SLOT_READERS = D == 64 ? EPI_WARPS : 4;
    static_assert(!(D == 256) || PAIR, "head_dim 256 needs the paired form to fit in shared memory");
    static_assert(SMEM <= 232448, "shared memory budget");
};

struct MmaParams {
    const float* vec;        // fp32 [U*Hq][D]: diag(Sigma_bar)/(2d)
    const uint8_t* image;    // bf16 images, IMG_FULL bytes per (unit, kv head, head subset)
    float* logits;           // fp32 [U, Hq, n]
    float* lse_part;         // fp32 [U*Hq][n_chunks (x2 for CTA pairs)][2]: (max, sum of exp) per work unit and CTA
    int* status;             // device-visible status word
    int Hq, Hkv, n;
    int n_subsets;           // head subsets per KV head
    int n_tiles;             // steps per head (128 keys per step, 256 with PAIR)
    int chunk_tiles;         // steps per work unit
    int n_chunks;            // work units per (unit, kv head)
    int n_groups;            // groups of n_subsets workers; a group walks a contiguous range of work units
    long long n_work;        // work units in all: (unit, kv head, chunk)
};

// ------------------------------------------------------------------------------------------
// Covariance image and epilogue vectors.  One CTA per query head.
template <int D>
__global__ void __launch_bounds__(256)
sigma_image_kernel(const ea_quad_form form, int Hq, int Hkv, uint8_t* __restrict__ image,
                   float* __restrict__ vec) {
    using G = Geo<D, true>;
    const int uh = blockIdx.x;
    const int u = uh / Hq, h = uh % Hq;
    const int Gq = Hq / Hkv;
    const int g = h / Gq, hg = h % Gq;
    const int n_subsets = (Gq + G::HPC - 1) / G::HPC;
    const int hs = hg / G::HPC, j = hg % G::HPC;
    const size_t set_head = (size_t)(u / form.units_per_set) * Hq + h;
    const float* S = form.quad + set_head * D * D;
    uint8_t* img = image + ((size_t)(u * Hkv + g) * n_subsets + hs) * G::IMG_FULL;   // 16-byte aligned
    const float quad_scale = form.quad_scale;  // 1/(2d) for Eq. 7, a power of two: the scaling is exact
    // per-channel scales of quantised rows (1 when the rows are the real keys)
    const float* cs = form.ch_scale ? form.ch_scale + (size_t)(u * Hkv + g) * D : nullptr;

    // Image rows in blocks of 32: the block needs S[c][:] (its own rows) and S[:][c] (its columns).  The
    // columns go through shared memory, loaded as 128-byte row segments, so that every global sector
    // is fetched once; a strided read of the columns kept this kernel bound by the L1 tag rate.
    // Thread = (lane: row c of the block, warp: 16-byte unit of 8 consecutive a, stepping by 8 units).
    __shared__ float col_s[D][33];                     // col_s[a][c - c_blk] = S[a][c]
    const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
    for (int c_blk = 0; c_blk < D; c_blk += 32) {
        __syncthreads();                               // the previous block's readers are done
        for (int e = threadIdx.x; e < D * 8; e += 256) {
            const int a = e / 8, piece = e % 8;
            const float4 x = __ldg(reinterpret_cast<const float4*>(S + (size_t)a * D + c_blk) + piece);
            col_s[a][4 * piece + 0] = x.x;
            col_s[a][4 * piece + 1] = x.y;
            col_s[a][4 * piece + 2] = x.z;
            col_s[a][4 * piece + 3] = x.w;
        }
        __syncthreads();
        const int c = c_blk + lane;
        const int row = G::col(j, c);
        const float s_c = cs ? cs[c] : 1.f;
        for (int a0 = warp * 8; a0 < D; a0 += 64) {
            const float4 r0 = __ldg(reinterpret_cast<const float4*>(S + (size_t)c * D + a0));
            const float4 r1 = __ldg(reinterpret_cast<const float4*>(S + (size_t)c * D + a0) + 1);
            const float own[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
            uint32_t w[4];
#pragma unroll
            for (int p = 0; p < 4; ++p) {
                uint32_t half[2];
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int a = a0 + 2 * p + q;
                    float val = 0.f;
                    if (a != c) {
                        // the two mirrored entries together carry (S_ca + S_ac) * quad_scale, split into a
                        // bf16 and the bf16 rounding of its remainder
                        const float s_ac = cs ? s_c * cs[a] : 1.f;
                        const float x = (own[2 * p + q] + col_s[a][lane]) * quad_scale * s_ac;
                        const float hi = __bfloat162float(__float2bfloat16_rn(x));
                        val = a < c ? hi : x - hi;
                    } else if (G::DIAG_MMA) {
                        val = own[2 * p + q] * quad_scale * s_c * s_c;   // its bf16 part; the rest in the diagonal blocks
                    }
                    half[q] = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(val));
                }
                w[p] = half[0] | (half[1] << 16);
            }
            const int kc = a0 / 64, unit = (a0 % 64) / 8;
            uint4* dst = reinterpret_cast<uint4*>(img + (size_t)kc * G::CHUNK_B_FULL + (size_t)row * 128 +
                                                  ((unit ^ (row & 7)) << 4));
            *dst = make_uint4(w[0], w[1], w[2], w[3]);
        }
    }
    // linear-term operand: row (j, c) holds mu_bar_c / sqrt(d) as a bf16 and the bf16 of its remainder in
    // K columns 0 and 1, zeros elsewhere; unswizzled core-matrix layout (8 rows x 16 bytes, K columns
    // 8..15 another 128 bytes on, next 8 rows 256 bytes on)
    for (int c = threadIdx.x; c < D; c += blockDim.x) {
        const float sc = cs ? cs[c] : 1.f;
        const float m = form.lin ? form.lin[set_head * D + c] * form.lin_scale * sc : 0.f;
        const __nv_bfloat16 hi = __float2bfloat16_rn(m);
        const __nv_bfloat16 lo = __float2bfloat16_rn(m - __bfloat162float(hi));
        const int row = G::col(j, c);
        uint8_t* dst = img + G::IMG_MAIN + (size_t)(row / 8) * 256 + (row % 8) * 16;
        *reinterpret_cast<uint4*>(dst) =
            make_uint4((uint32_t)__bfloat16_as_ushort(hi) | ((uint32_t)__bfloat16_as_ushort(lo) << 16), 0u, 0u, 0u);
        *reinterpret_cast<uint4*>(dst + 128) = make_uint4(0u, 0u, 0u, 0u);
        const float dg = S[(size_t)c * D + c] * quad_scale * sc * sc;
        vec[(size_t)uh * D + c] = dg;
        if (G::DIAG_MMA) {
            // block c / 16 (one per MMA step), row n = 16 j + c % 16, K column c % 16: the bf16 of what the
            // image's diagonal entry left of dg; zeros elsewhere in the row
            const __nv_bfloat16 lo = __float2bfloat16_rn(dg - __bfloat162float(__float2bfloat16_rn(dg)));
            const int kk = c % 16, n = 16 * j + kk;
            uint8_t* blk = img + G::IMG_MAIN + G::LIN_FULL + (size_t)(c / 16) * G::DIAG_BLOCK +
                           (n / 8) * 256 + (n % 8) * 16;
            uint32_t w4[4] = {0u, 0u, 0u, 0u};
            w4[(kk % 8) / 2] = (uint32_t)__bfloat16_as_ushort(lo) << (16 * (kk % 2));
            const uint4 mine = make_uint4(w4[0], w4[1], w4[2], w4[3]), zero = make_uint4(0u, 0u, 0u, 0u);
            *reinterpret_cast<uint4*>(blk) = kk < 8 ? mine : zero;            // K columns 0..7
            *reinterpret_cast<uint4*>(blk + 128) = kk < 8 ? zero : mine;      // K columns 8..15
        }
    }
}

// ------------------------------------------------------------------------------------------
struct Item {
    int ug, hs, tile0, tile1, hpc;
};

// Work unit w of head subset hs: a run of key tiles of one (unit, kv head).  The workers of a group
// (one per head subset) walk the same units at the same time, so the key tiles they share are
// fetched from HBM once, and a worker changes its covariance image only when the head changes.
__device__ __forceinline__ Item decode_item(long long w, int hs, const MmaParams& p, int hpc_max) {
    Item it;
    it.hs = hs;
    const int chunk = (int)(w % p.n_chunks);
    it.ug = (int)(w / p.n_chunks);
    it.tile0 = chunk * p.chunk_tiles;
    it.tile1 = min(p.n_tiles, it.tile0 + p.chunk_tiles);
    const int Gq = p.Hq / p.Hkv;
    it.hpc = min(hpc_max, Gq - it.hs * hpc_max);
    return it;
}

// Four E4M3 codes (one per byte of w, lowest channel in the lowest byte) -> four bf16, exact.  A code
// s eeee mmm is laid out as the bf16 pattern s 0000eeee mmm0000, which reads (-1)^s 2^(e-127) (1 + m/8) or,
// for e = 0, the bf16 subnormal (-1)^s 2^-126 m/8; times 2^120 that is the E4M3 value in either case
// (bias 7, subnormals m 2^-9).  The byte permute also spreads the sign over the byte above each code, so
// one shift and one mask place all three fields.  The NaN codes 0x7f and 0xff have no place in a cache and
// read as +-480 here.
__device__ __forceinline__ void e4m3x4_to_bf16x4(uint32_t w, uint32_t& lo, uint32_t& hi) {
    uint32_t a, b;
    asm("prmt.b32 %0, %1, 0, 0x9180;" : "=r"(a) : "r"(w));       // (sign(b1), b1, sign(b0), b0)
    asm("prmt.b32 %0, %1, 0, 0xb3a2;" : "=r"(b) : "r"(w));       // (sign(b3), b3, sign(b2), b2)
    a = (a << 4) & 0x87f087f0u;
    b = (b << 4) & 0x87f087f0u;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(lo) : "r"(a), "r"(0x7b807b80u));   // x 2^120
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(hi) : "r"(b), "r"(0x7b807b80u));
}

// AND of `ok` over the NT threads that meet at named barrier ID: keeps their control flow identical.
template <int ID, int NT>
__device__ __forceinline__ bool named_all(bool ok) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.b32 q, %1, 0;\n\t"
        "bar.red.and.pred p, %2, %3, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"((uint32_t)ok), "n"(ID), "n"(NT)
        : "memory");
    return r != 0;
}
// the epilogue threads' barrier
template <int NT>
__device__ __forceinline__ bool epi_all(bool ok) { return named_all<1, NT>(ok); }

template <int D, bool PAIR, bool Q8>
__global__ void __launch_bounds__(Geo<D, PAIR, Q8>::THREADS, 1)
logits_mma_kernel(const __grid_constant__ CUtensorMap k_map, const MmaParams p) {
    using G = Geo<D, PAIR, Q8>;
    static_assert(!(G::DIAG_MMA && PAIR), "the diagonal blocks are laid out for a single CTA");
    extern __shared__ uint8_t smem_raw[];
    // carve shared memory: 1024-byte aligned operand tiles first
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    uint8_t* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const uint32_t s_img = base;
    const uint32_t s_k = s_img + G::IMG_CTA;
    constexpr int kOffOnes = G::IMG_CTA + G::NSLOT * kChunkA;
    const uint32_t s_ones = base + kOffOnes;
    const uint32_t s_lin = s_ones + G::ONES;
    constexpr int kOffVec = kOffOnes + G::ONES + G::LIN_CTA;
    const uint32_t s_vec = base + kOffVec;                       // fp32 diagonals (d = 256)
    const uint32_t s_diag = s_vec + G::VEC;        // 16 x 16 diagonal blocks (d <= 128)
    constexpr int kOffPart = kOffVec + G::VEC + G::DIAG_FULL;
    float* part_gen = reinterpret_cast<float*>(gen_base + kOffPart);
    float* red_gen = reinterpret_cast<float*>(gen_base + kOffPart + G::PART);
    const uint32_t s_bar = base + kOffPart + G::PART + G::RED;
    uint8_t* bar_gen = gen_base + kOffPart + G::PART + G::RED;
    // per ring slot: the chunk has landed / its readers are done with it
    auto full_k = [&](int slot) { return s_bar + 8u * slot; };
    auto empty_k = [&](int slot) { return s_bar + 8u * (G::NSLOT + slot); };
    auto tmem_full = [&](int a) { return s_bar + 8u * (2 * G::NSLOT + a); };
    auto tmem_empty = [&](int a) { return s_bar + 8u * (2 * G::NSLOT + 2 + a); };
    const uint32_t img_full = s_bar + 8u * (2 * G::NSLOT + 4);
    const uint32_t img_peer = s_bar + 8u * (2 * G::NSLOT + 5);
    auto q_full = [&](int slot) { return s_bar + 8u * (2 * G::NSLOT + 6 + slot); };     // Q8: the slot's codes have landed
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_gen + 8 * G::NBAR);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_gen + 8 * G::NBAR + 4);

    const int warp = threadIdx.x / 32, lane = threadIdx.x % 32;
    const uint32_t rank = PAIR ? cluster_ctarank() : 0u;     // 0 = leader
    const bool leader = rank == 0;

    if (threadIdx.x == 0) {
        for (int s = 0; s < G::NSLOT; ++s) {
            mbar_init(full_k(s), G::FILLERS);                      // Q8: the widening warps fill the slot
            mbar_init(empty_k(s), G::SLOT_READERS);
        }
        for (int s = 0; s < G::NQ; ++s) mbar_init(q_full(s), 1);
        for (int a = 0; a < 2; ++a) {
            mbar_init(tmem_full(a), 1);
            mbar_init(tmem_empty(a), PAIR ? 2 * G::EPI_WARPS : G::EPI_WARPS);
        }
        mbar_init(img_full, 1);
        mbar_init(img_peer, 1);
        *abort_flag = 0;
        fence_mbar_init();
        prefetch_tensormap(&k_map);
    }
    // constant A operand of the linear-term step: K columns 0 and 1 are one, the rest zero
    // (row r of the tile at (r / 8) * 256 + (r % 8) * 16, K columns 8..15 another 128 bytes on)
    for (int e = threadIdx.x; e < G::ONES / 16; e += G::THREADS) {
        const int piece = e % 16;                       // 16-byte pieces of a 256-byte group of 8 rows
        uint4 v = make_uint4(piece < 8 ? 0x3f803f80u : 0u, 0u, 0u, 0u);   // two bf16 ones, then zeros
        *reinterpret_cast<uint4*>(gen_base + kOffOnes + e * 16) = v;
    }
    fence_proxy_async_smem();
    if (warp == 1) {
        if (PAIR) {
            tmem_alloc_pair(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
            tmem_relinquish_pair();
        } else {
            tmem_alloc(smem_u32(const_cast<uint32_t*>(tmem_slot)), kTmemCols);
            tmem_relinquish();
        }
    }
    tc_fence_before_sync();
    __syncthreads();
    if (PAIR) cluster_sync();          // the peer's barriers exist before anything signals them
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_slot;

    const int worker = PAIR ? blockIdx.x / 2 : blockIdx.x;
    const int my_hs = worker % p.n_subsets;
    const long long my_group = worker / p.n_subsets;
    const long long first = p.n_work * my_group / p.n_groups;
    const long long last = p.n_work * (my_group + 1) / p.n_groups;
    constexpr int kKeysPerStep = PAIR ? 2 * kTileKeys : kTileKeys;
    // Chunk number c = tile_no * KCH + kc of this worker's stream of key tiles lives in ring slot
    // c % NSLOT, on its (c / NSLOT)-th use.
    auto slot_of = [](long long c) { return (int)(c % G::NSLOT); };
    auto use_of = [](long long c) { return (uint32_t)(c / G::NSLOT); };

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0) {
            long long tile_no = 0, cur_img = -1, issued = 0;      // issued: chunks whose copy has been started
            bool ok = true;
            for (long long item = first; ok && item < last; ++item) {
                const Item it = decode_item(item, my_hs, p, G::HPC);
                const long long img_id = (long long)it.ug * p.n_subsets + it.hs;
                if (img_id != cur_img) {
                    // Every chunk that used the resident image must have been handed back: the epilogue warps
                    // that release a slot only run after the tile's MMAs, and by the time a warp releases its
                    // last chunk of a tile it has also read the last of the image's diagonal.
                    for (int back = 1; ok && back <= G::NSLOT && back <= issued; ++back) {
                        const long long c = issued - back;
                        ok = mbar_wait(empty_k(slot_of(c)), use_of(c) & 1, abort_flag);
                    }
                    if (!ok) break;
                    const int rows_total = (G::DIAG_MMA ? G::HPC : it.hpc) * D;     // interleaved heads: every row
                    const int rows = PAIR ? rows_total / 2 : rows_total;
                    const int u = it.ug / p.Hkv, g = it.ug % p.Hkv;
                    const int h0 = g * (p.Hq / p.Hkv) + it.hs * G::HPC;
                    // the fp32 diagonal for the epilogue (d = 256) or the diagonal blocks for the tensor cores
                    const uint32_t vec_bytes = G::DIAG_MMA ? (uint32_t)G::DIAG_FULL
                                                           : (uint32_t)(it.hpc * D * sizeof(float));
                    mbar_arrive_expect_tx(img_full, (uint32_t)(G::KCH * rows * 128 + rows * 32) + vec_bytes);
                    const uint8_t* img = p.image + (size_t)img_id * G::IMG_FULL;
                    const uint8_t* src = img + (size_t)rank * rows * 128;
                    for (int kc = 0; kc < G::KCH; ++kc)
                        bulk_load(s_img + kc * G::CHUNK_B, src + (size_t)kc * G::CHUNK_B_FULL, rows * 128, img_full);
                    bulk_load(s_lin, img + G::IMG_MAIN + (size_t)rank * rows * 32, rows * 32, img_full);
                    if (G::DIAG_MMA) bulk_load(s_diag, img + G::IMG_MAIN + G::LIN_FULL, vec_bytes, img_full);
                    else bulk_load(s_vec, p.vec + ((size_t)u * p.Hq + h0) * D, vec_bytes, img_full);
                    cur_img = img_id;
                }
                for (int t = it.tile0; ok && t < it.tile1; ++t, ++tile_no) {
                    const int key0 = t * kKeysPerStep + (int)rank * kTileKeys;
                    for (int kc = 0; ok && kc < G::KCH; ++kc) {
                        const long long c = tile_no * G::KCH + kc;
                        const int slot = slot_of(c);
                        ok = mbar_wait(empty_k(slot), (use_of(c) & 1) ^ 1, abort_flag);
                        if (!ok) break;
                        if constexpr (Q8) {
                            // codes go to the upper half of the slot; the widening warps spread them over it
                            mbar_arrive_expect_tx(q_full(slot), kChunkQ);
                            tma_load_3d(s_k + slot * kChunkA + kChunkQ, &k_map, q_full(slot), kc * 64, key0, it.ug);
                            issued = c + 1;
                            continue;
                        }
                        if (PAIR) {
                            // both CTAs' copies are counted on the leader's barrier, which the MMA issuer watches
                            if (leader) mbar_arrive_expect_tx(full_k(slot), 2 * kChunkA);
                            tma_load_3d_pair(s_k + slot * kChunkA, &k_map, mapa(full_k(slot), 0), kc * 64, key0,
                                             it.ug);
                        } else {
                            mbar_arrive_expect_tx(full_k(slot), kChunkA);
                            tma_load_3d(s_k + slot * kChunkA, &k_map, full_k(slot), kc * 64, key0, it.ug);
                        }
                        issued = c + 1;
                    }
                }
            }
            if (!ok && Q8) {
                for (int back = 1; back <= G::NSLOT && back <= issued; ++back) {
                    const long long c = issued - back;
                    mbar_drain(q_full(slot_of(c)), use_of(c) & 1);
                }
            } else if (!ok && leader) {
                // Let the copies already in flight land before the shared memory goes away.  In a pair the
                // leader's barriers count both CTAs' bytes, and the peer stays until the teardown's cluster
                // barrier, which the leader reaches only after this.  Bounded by time: a copy the peer
                // never started is not waited for beyond that.
                for (int back = 1; back <= G::NSLOT && back <= issued; ++back) {
                    const long long c = issued - back;
                    mbar_drain(full_k(slot_of(c)), use_of(c) & 1);
                }
            }
        }
        __syncwarp();
    } else if (warp == 1) {
        if (lane == 0 && leader) {
            // -------------------------------------------------------------- MMA issuer
            long long tile_no = 0, cur_img = -1;
            int img_loads = 0;
            bool ok = true;
            for (long long item = first; ok && item < last; ++item) {
                const Item it = decode_item(item, my_hs, p, G::HPC);
                const long long img_id = (long long)it.ug * p.n_subsets + it.hs;
                if (img_id != cur_img) {
                    ok = mbar_wait(img_full, img_loads & 1, abort_flag);
                    if (ok && PAIR) ok = mbar_wait<true>(img_peer, img_loads & 1, abort_flag);
                    if (!ok) break;
                    ++img_loads;
                    cur_img = img_id;
                }
                // (interleaved heads: a pass with fewer heads still spans every column; the columns of the
                // missing heads hold whatever the image rows held and are never read)
                const uint32_t n_cols = (uint32_t)((G::DIAG_MMA ? G::HPC : it.hpc) * D);
                const uint32_t idesc = PAIR ? umma_idesc_bf16_m256(n_cols) : umma_idesc_bf16_m128(n_cols);
                for (int t = it.tile0; ok && t < it.tile1; ++t, ++tile_no) {
                    const int a = (int)(tile_no & 1);
                    const uint32_t use = (uint32_t)(tile_no >> 1);
                    ok = mbar_wait<PAIR>(tmem_empty(a), (use & 1) ^ 1, abort_flag);
                    if (!ok) break;
                    tc_fence_after_sync();
                    const uint32_t d_tmem = tmem_base + (uint32_t)(a * kAccCols);
                    {   // linear term first, overwriting the stage: D = ones . (hi, lo of mu')^T
                        const uint64_t da = umma_desc_k_plain(s_ones);
                        const uint64_t db = umma_desc_k_plain(s_lin);
                        if (PAIR) umma_bf16_pair(d_tmem, da, db, idesc, 0u);
                        else umma_bf16(d_tmem, da, db, idesc, 0u);
                    }
#pragma unroll
                    for (int kc = 0; kc < G::KCH; ++kc) {
                        const long long c = tile_no * G::KCH + kc;
                        const int slot = slot_of(c);
                        ok = ok && mbar_wait<PAIR>(full_k(slot), use_of(c) & 1, abort_flag);
                        if (!ok) break;
                        tc_fence_after_sync();
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks) {
                            const uint64_t da = umma_desc_k_sw128(s_k + slot * kChunkA + ks * 32);
                            const uint64_t db = umma_desc_k_sw128(s_img + kc * G::CHUNK_B + ks * 32);
                            if (PAIR) umma_bf16_pair(d_tmem, da, db, idesc, 1u);
                            else umma_bf16(d_tmem, da, db, idesc, 1u);
                        }
                    }
                    if (!ok) break;
                    if (G::DIAG_MMA) {
                        // D[:, c] += k_c * lo(diag_c) for every head: one N = 16 HPC step per 16 channels
                        const uint32_t idesc_d = umma_idesc_bf16_m128(16 * G::HPC);
#pragma unroll
                        for (int ks = 0; ks < D / 16; ++ks) {
                            const int slot = slot_of(tile_no * G::KCH + ks / 4);
                            umma_bf16(d_tmem + (uint32_t)(ks * 16 * G::HPC),
                                      umma_desc_k_sw128(s_k + slot * kChunkA + (ks % 4) * 32),
                                      umma_desc_k_plain(s_diag + (uint32_t)(ks * G::DIAG_BLOCK)), idesc_d, 1u);
                        }
                    }
                    if (PAIR) umma_commit_pair(tmem_full(a), 3);
                    else umma_commit(tmem_full(a));
                }
            }
        } else if (PAIR && lane == 0) {
            // ---------------------------------------------- peer: report each landed image half
            long long cur_img = -1;
            int img_loads = 0;
            bool ok = true;
            for (long long item = first; ok && item < last; ++item) {
                const Item it = decode_item(item, my_hs, p, G::HPC);
                const long long img_id = (long long)it.ug * p.n_subsets + it.hs;
                if (img_id != cur_img) {
                    ok = mbar_wait(img_full, img_loads & 1, abort_flag);
                    if (!ok) break;
                    mbar_arrive_cluster(mapa(img_peer, 0));
                    ++img_loads;
                    cur_img = img_id;
                }
            }
        }
        __syncwarp();
    } else if (warp >= 2 + G::EPI_WARPS) {
        // ------------------------------------------------------------------ code -> bf16 (Q8)
        // 512 pieces of 16 codes per chunk: thread t takes pieces t, t + 128, ... (a warp reads
        // 512 contiguous bytes); piece (row, u) becomes the 16-byte units 2u and 2u + 1 of the row's 128
        // bytes in the slot, at the swizzled places the MMA and the epilogue expect.  The bf16 rows cover the
        // codes they came from, so every thread holds its codes in registers before any thread writes.
        const int ct = threadIdx.x - 32 * (2 + G::EPI_WARPS);
        constexpr int kConvThreads = 32 * (G::CONV_WARPS > 0 ? G::CONV_WARPS : 1);
        constexpr int kPieces = kChunkQ / 16 / kConvThreads;          // 16-code pieces per thread and chunk
        long long tile_no = 0;
        bool ok = true;
        for (long long item = first; ok && item < last; ++item) {
            const Item it = decode_item(item, my_hs, p, G::HPC);
            for (int t = it.tile0; ok && t < it.tile1; ++t, ++tile_no) {
                for (int kc = 0; ok && kc < G::KCH; ++kc) {
                    const long long c = tile_no * G::KCH + kc;
                    const int slot = slot_of(c);
                    bool my_ok = mbar_wait(q_full(slot), use_of(c) & 1, abort_flag);
                    const uint32_t dst = s_k + slot * kChunkA, src = dst + kChunkQ;
                    uint4 x[kPieces];
                    if (my_ok) {
#pragma unroll
                        for (int i = 0; i < kPieces; ++i) x[i] = lds128(src + (ct + kConvThreads * i) * 16);
                    }
                    // named barrier 2: all codes are in registers (and a wait that gave up stops all four warps)
                    if (!named_all<2, kConvThreads>(my_ok)) {
                        ok = false;
                        break;
                    }
#pragma unroll
                    for (int i = 0; i < kPieces; ++i) {
                        const int piece = ct + kConvThreads * i, r = piece / 4, u = piece % 4;
                        uint32_t o[8];
                        e4m3x4_to_bf16x4(x[i].x, o[0], o[1]);
                        e4m3x4_to_bf16x4(x[i].y, o[2], o[3]);
                        e4m3x4_to_bf16x4(x[i].z, o[4], o[5]);
                        e4m3x4_to_bf16x4(x[i].w, o[6], o[7]);
                        sts128(dst + r * 128 + (((2 * u) ^ (r & 7)) << 4), make_uint4(o[0], o[1], o[2], o[3]));
                        sts128(dst + r * 128 + (((2 * u + 1) ^ (r & 7)) << 4), make_uint4(o[4], o[5], o[6], o[7]));
                    }
                    fence_proxy_async_smem();          // the MMA reads these bytes through the async proxy
                    __syncwarp();
                    if (lane == 0) {
                        // In a pair the leader's barrier counts both CTAs' widening warps.  The bytes stay on
                        // this SM (its own tensor core reads them) and the proxy fence above has completed the
                        // stores, so the plain remote arrival is enough; a cluster-wide release here stalls the
                        // warp for about a microsecond per chunk and doubled the kernel's time.
                        if (PAIR) mbar_arrive_cluster(mapa(full_k(slot), 0));
                        else mbar_arrive(full_k(slot));
                    }
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ epilogue
        // Warp (quarter, part): accumulator lanes 32*quarter.. (thread <-> lane <-> key) and columns
        // [part * CPP, (part + 1) * CPP) of every head of the pass.  The parts of a key meet in shared
        // memory and are added in part order; head j is finished and stored by part j % EPI_PARTS.
        const int ew = warp - 2;
        const int quarter = warp % 4;              // the TMEM lanes this warp may read
        const int cp = ew / 4;                     // column part
        const int row = quarter * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        // accumulator columns per tensor-memory load; the widening warps cap the kernel at 128 registers, which
        // the 32-column form of head_dim 256 does not fit
        constexpr int BW = (D == 256 && !Q8) ? 32 : 16;
        constexpr int NBW = (G::CPP / BW) * G::HPC;                 // loads per tile for this warp
        constexpr int kEpiThreads = 32 * G::EPI_WARPS;
        const uint32_t empty_remote = PAIR ? mapa(tmem_empty(0), 0) : 0u;
        long long tile_no = 0, cur_img = -1;
        int img_loads = 0;
        bool ok = true;
        for (long long item = first; ok && item < last; ++item) {
            const Item it = decode_item(item, my_hs, p, G::HPC);
            const long long img_id = (long long)it.ug * p.n_subsets + it.hs;
            bool img_ok = true;
            if (img_id != cur_img) {
                img_ok = mbar_wait(img_full, img_loads & 1, abort_flag);
                ++img_loads;
                cur_img = img_id;
            }
            const int u = it.ug / p.Hkv, g = it.ug % p.Hkv;
            const int h0 = g * (p.Hq / p.Hkv) + it.hs * G::HPC;
            // running (max, sum of exp) of this thread's keys, for the heads this part finishes
            float m_run[G::HPC], l_run[G::HPC];
#pragma unroll
            for (int j = 0; j < G::HPC; ++j) { m_run[j] = -INFINITY; l_run[j] = 0.f; }
            for (int t = it.tile0; ok && t < it.tile1; ++t, ++tile_no) {
                const int a = (int)(tile_no & 1);
                const long long c_tile = tile_no * G::KCH;
                bool my_ok = img_ok;
                my_ok = my_ok && mbar_wait<PAIR>(tmem_full(a), (uint32_t)((tile_no >> 1) & 1), abort_flag);
                my_ok = __all_sync(0xffffffffu, my_ok);
                float* part = part_gen + (tile_no & 1) * (G::EPI_PARTS * G::HPC * kTileKeys);
                if (my_ok) {
                    tc_fence_after_sync();
                    float2 acc[G::HPC][2];
#pragma unroll
                    for (int j = 0; j < G::HPC; ++j) acc[j][0] = acc[j][1] = make_float2(0.f, 0.f);
                    // load b -> (columns c0 .. c0 + BW of head j): heads innermost so the unpacked key values
                    // are reused.  Narrow loads at d <= 128, where the epilogue is the limit: few live registers
                    // leave the scheduler room to overlap the dependent FMAs.
                    auto c0_of = [&](int b) { return cp * G::CPP + (b / G::HPC) * BW; };
                    auto addr_of = [&](int b) {
                        return t_lane + (uint32_t)(a * kAccCols + G::col(b % G::HPC, c0_of(b)));
                    };
                    uint32_t dv[2][BW];
                    tmem_ld_cols(addr_of(0), dv[0]);      // head 0 always exists
                    float2 kf[BW / 2];
#pragma unroll
                    for (int b = 0; b < NBW; ++b) {
                        const int j = b % G::HPC;
                        const int c0 = c0_of(b);
                        if (j == 0) {
                            const uint32_t k_row = s_k + slot_of(c_tile + c0 / 64) * kChunkA + row * 128;
#pragma unroll
                            for (int q = 0; q < BW / 8; ++q) {
                                const int unit = (c0 % 64) / 8 + q;
                                const uint4 w = lds128(k_row + ((unit ^ (row & 7)) << 4));
                                const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
                                for (int e = 0; e < 4; ++e)
                                    kf[q * 4 + e] = make_float2(__uint_as_float(ww[e] << 16),
                                                                __uint_as_float(ww[e] & 0xffff0000u));
                            }
                        }
                        // the block's diagonal constants, requested before the accumulator wait so that
                        // their latency is not paid inside the arithmetic
                        uint4 dgv[BW / 4];
                        if (!G::DIAG_MMA && j < it.hpc) {
#pragma unroll
                            for (int q = 0; q < BW / 4; ++q) dgv[q] = lds128(s_vec + (uint32_t)((j * D + c0 + 4 * q) * 4));
                        }
                        tmem_ld_wait();
                        if (b + 1 < NBW && (b + 1) % G::HPC < it.hpc) tmem_ld_cols(addr_of(b + 1), dv[(b + 1) & 1]);
                        if (j < it.hpc) {
                            // accumulator = K.B^T + mu' (the linear term rode in on the extra MMA step)
                            const uint32_t* dd = dv[b & 1];
#pragma unroll
                            for (int q = 0; q < BW / 4; ++q) {
                                const float2 k0 = kf[2 * q], k1 = kf[2 * q + 1];
                                if (G::DIAG_MMA) {
                                    // the whole bracket came from the tensor cores: one FMA per element
                                    acc[j][0] = fma2(k0, make_float2(__uint_as_float(dd[4 * q]), __uint_as_float(dd[4 * q + 1])),
                                                     acc[j][0]);
                                    acc[j][1] = fma2(k1, make_float2(__uint_as_float(dd[4 * q + 2]), __uint_as_float(dd[4 * q + 3])),
                                                     acc[j][1]);
                                    continue;
                                }
                                const float4 dg = make_float4(__uint_as_float(dgv[q].x), __uint_as_float(dgv[q].y),
                                                              __uint_as_float(dgv[q].z), __uint_as_float(dgv[q].w));
                                const float2 t0 = fma2(make_float2(dg.x, dg.y), k0,
                                                       make_float2(__uint_as_float(dd[4 * q]), __uint_as_float(dd[4 * q + 1])));
                                const float2 t1 = fma2(make_float2(dg.z, dg.w), k1,
                                                       make_float2(__uint_as_float(dd[4 * q + 2]), __uint_as_float(dd[4 * q + 3])));
                                acc[j][0] = fma2(k0, t0, acc[j][0]);
                                acc[j][1] = fma2(k1, t1, acc[j][1]);
                            }
                        }
                        // hand the 64-channel chunk back to the producer once this warp is done with it
                        const bool chunk_done = j == G::HPC - 1 && (D == 64 ? b == NBW - 1 : (c0 + BW) % 64 == 0);
                        if (chunk_done) {
                            __syncwarp();
                            if (lane == 0) mbar_arrive(empty_k(slot_of(c_tile + c0 / 64)));
                        }
                    }
                    // the accumulator stage is free again
                    tc_fence_before_sync();
                    __syncwarp();
                    if (lane == 0) {
                        if (PAIR && !leader) mbar_arrive_cluster(empty_remote + 8u * a);
                        else mbar_arrive(tmem_empty(a));
                    }
#pragma unroll
                    for (int j = 0; j < G::HPC; ++j)
                        part[(cp * G::HPC + j) * kTileKeys + row] =
                            (acc[j][0].x + acc[j][1].x) + (acc[j][0].y + acc[j][1].y);
                }
                // one named barrier per tile: the parts exchange their partial sums, and a wait
                // that gave up anywhere stops every epilogue warp at the same tile
                if (!epi_all<kEpiThreads>(my_ok)) {
                    ok = false;
                    break;
                }
                const int key = t * kKeysPerStep + (int)rank * kTileKeys + row;
                if (key < p.n) {
#pragma unroll
                    for (int j = 0; j < G::HPC; ++j)
                        if (j % G::EPI_PARTS == cp && j < it.hpc) {
                            float sv = part[j * kTileKeys + row];
#pragma unroll
                            for (int q = 1; q < G::EPI_PARTS; ++q) sv += part[(q * G::HPC + j) * kTileKeys + row];
                            p.logits[((size_t)u * p.Hq + h0 + j) * (size_t)p.n + key] = sv;
                            const float m_new = fmaxf(m_run[j], sv);
                            l_run[j] = l_run[j] * __expf(m_run[j] - m_new) + __expf(sv - m_new);
                            m_run[j] = m_new;
                        }
                }
            }
            if (!ok) break;
            // log-sum-exp partial of the work unit: lanes, then the four warps of the finishing part
#pragma unroll
            for (int j = 0; j < G::HPC; ++j)
                if (j % G::EPI_PARTS == cp) {
                    float m = m_run[j], l = l_run[j];
#pragma unroll
                    for (int off = 16; off > 0; off >>= 1) {
                        const float mo = __shfl_xor_sync(0xffffffffu, m, off);
                        const float lo = __shfl_xor_sync(0xffffffffu, l, off);
                        const float mn = fmaxf(m, mo);
                        l = mn == -INFINITY ? 0.f : l * __expf(m - mn) + lo * __expf(mo - mn);
                        m = mn;
                    }
                    if (lane == 0) {
                        red_gen[(j * 4 + quarter) * 2 + 0] = m;
                        red_gen[(j * 4 + quarter) * 2 + 1] = l;
                    }
                }
            if (!epi_all<kEpiThreads>(true)) { ok = false; break; }
            if (threadIdx.x - 64 < G::HPC && (int)(threadIdx.x - 64) < it.hpc) {
                const int j = threadIdx.x - 64;
                float m = -INFINITY, l = 0.f;
                for (int w = 0; w < 4; ++w) {          // fixed order: bitwise reproducible
                    const float mo = red_gen[(j * 4 + w) * 2], lo = red_gen[(j * 4 + w) * 2 + 1];
                    const float mn = fmaxf(m, mo);
                    l = mn == -INFINITY ? 0.f : l * __expf(m - mn) + lo * __expf(mo - mn);
                    m = mn;
                }
                // one slot per work unit and CTA of the pair
                constexpr int R = PAIR ? 2 : 1;
                const int slot = (int)(item % p.n_chunks) * R + (int)rank;
                float* dst = p.lse_part + (((size_t)u * p.Hq + h0 + j) * (p.n_chunks * R) + slot) * 2;
                dst[0] = m;
                dst[1] = l;
            }
        }
    }

    // ---------------------------------------------------------------------- teardown
    tc_fence_before_sync();
    __syncthreads();
    if (PAIR) cluster_sync();          // the peer may still read this CTA's shared memory until here
    if (warp == 1) {
        tc_fence_after_sync();
        if (PAIR) tmem_dealloc_pair(tmem_base, kTmemCols);
        else tmem_dealloc(tmem_base, kTmemCols);
    }
    if (threadIdx.x == 0 && *abort_flag) *p.status = (int)EA_ERR_DEVICE_TIMEOUT;
}

// ------------------------------------------------------------------------------------------
// K as a rank-3 tensor (d, n, unit*kv_head); one box is 64 channels x 128 keys, 128-byte swizzle.
// Rows past n read as zero; heads are kv_capacity rows apart.
bool make_k_map(CUtensorMap* map, const void* k, int d, int n, int cap, long long heads, bool codes) {
    const uint64_t es = codes ? 1 : 2;                 // bytes per element: FP8 codes or bf16
    return ea_tensor_map_bf16_3d(map, k, (uint64_t)d, (uint64_t)n, (uint64_t)heads, (uint64_t)d * es,
                                 (uint64_t)cap * d * es, 64, kTileKeys, codes);
}

template <int D, bool PAIR, bool Q8>
ea_status launch_mma(const ea_ctx* ctx, const ea_shape& s, const void* k, const ea_quad_form& form,
                     uint8_t* image, float* vec, float* logits, float* lse_part, int* n_chunks_out,
                     cudaStream_t st) {
    using G = Geo<D, PAIR, Q8>;
    const int Gq = s.n_q_heads / s.n_kv_heads;
    constexpr int keys_per_step = PAIR ? 2 * kTileKeys : kTileKeys;
    // CTAs or CTA pairs, one per SM; the SMs of a side pass (ea_set_side_sms) are left to it
    const int sms = ctx->sm_budget < ctx->sm_count - ctx->side_sms ? ctx->sm_budget : ctx->sm_count - ctx->side_sms;
    const int workers = PAIR ? sms / 2 : sms;
    MmaParams p;
    p.vec = vec;
    p.image = image;
    p.logits = logits;
    p.lse_part = lse_part;
    p.status = ctx->status_dev;
    p.Hq = s.n_q_heads;
    p.Hkv = s.n_kv_heads;
    p.n = s.n_keys;
    p.n_subsets = (Gq + G::HPC - 1) / G::HPC;
    p.n_tiles = (s.n_keys + keys_per_step - 1) / keys_per_step;
    // Workers come in groups of n_subsets (one per head subset); every group gets an equal,
    // contiguous share of the work units, which are cut fine enough to balance the groups.
    const long long heads = (long long)s.n_units * s.n_kv_heads;
    p.n_groups = workers / p.n_subsets;
    if (p.n_groups < 1) return EA_ERR_UNSUPPORTED;
    if (p.n_groups > heads * p.n_tiles) p.n_groups = (int)(heads * p.n_tiles);
    int chunk = p.n_tiles;
    while (chunk > 4 && heads * ((p.n_tiles + chunk - 1) / chunk) < 32LL * p.n_groups) chunk = (chunk + 1) / 2;
    p.chunk_tiles = chunk;
    p.n_chunks = (p.n_tiles + chunk - 1) / chunk;
    p.n_work = heads * p.n_chunks;
    *n_chunks_out = p.n_chunks * (PAIR ? 2 : 1);

    CUtensorMap k_map;
    if (!make_k_map(&k_map, k, D, s.n_keys, ea_kv_cap(s), (long long)s.n_units * s.n_kv_heads, Q8)) return EA_ERR_CUDA;

    if (form.quad)
        sigma_image_kernel<D><<<s.n_units * s.n_q_heads, 256, 0, st>>>(form, s.n_q_heads, s.n_kv_heads, image, vec);
    auto kern = logits_mma_kernel<D, PAIR, Q8>;
    EA_CUDA_TRY(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, G::SMEM));
    const long long want = (long long)p.n_groups * p.n_subsets;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(PAIR ? 2 * want : want));
    cfg.blockDim = dim3(G::THREADS);
    cfg.dynamicSmemBytes = G::SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = PAIR ? 2 : 1;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ea_count_launches(ctx, form.quad ? 2 : 1);
    cudaEvent_t stop = ea_profile_mark_start(ctx, st);
    const cudaError_t err = cudaLaunchKernelEx(&cfg, kern, k_map, p);
    ea_profile_mark_stop(ctx, stop, st);
    EA_CUDA_TRY(err);
    return EA_CHECK_LAUNCH();
}

}  // namespace

// bf16 rank-3 tensor map (innermost extent first) with a (box0 x box1 x 1) box, 128-byte swizzle,
// zero fill outside the tensor.  Strides in bytes, multiples of 16; base 16-byte aligned.
bool ea_tensor_map_bf16_3d(CUtensorMap* map, const void* base, uint64_t n0, uint64_t n1, uint64_t n2,
                           uint64_t stride1, uint64_t stride2, uint32_t box0, uint32_t box1, bool bytes_plain) {
    typedef CUresult (*encode_tiled_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                        const cuuint64_t*, const cuuint32_t*, const cuuint32_t*,
                                        CUtensorMapInterleave, CUtensorMapSwizzle, CUtensorMapL2promotion,
                                        CUtensorMapFloatOOBfill);
    // resolved once, under std::call_once: first calls may come from several host threads
    static std::once_flag once;
    static encode_tiled_fn fn = nullptr;
    std::call_once(once, [] {
        void* ptr = nullptr;
        cudaDriverEntryPointQueryResult res;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &res) == cudaSuccess &&
            res == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<encode_tiled_fn>(ptr);
        else
            cudaGetLastError();
    });
    if (!fn) return false;
    const cuuint64_t dims[3] = {n0, n1, n2};
    const cuuint64_t strides[2] = {stride1, stride2};
    const cuuint32_t box[3] = {box0, box1, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    // bytes_plain: 8-bit elements, rows of the box stored one after the other without swizzle
    return fn(map, bytes_plain ? CU_TENSOR_MAP_DATA_TYPE_UINT8 : CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
              const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              bytes_plain ? CU_TENSOR_MAP_SWIZZLE_NONE : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool ea_mma_path_supported(const ea_shape& s) {
    // one worker (CTA or CTA pair) per head subset of a KV head must exist even on the smallest SM budget
    // (ea_set_sm_budget admits 32 SMs = 16 pairs); wider groups take the CUDA-core kernel
    const int subsets = (s.n_q_heads / s.n_kv_heads + 256 / s.head_dim - 1) / (256 / s.head_dim);
    if (subsets > 16) return false;
    if (s.head_dim == 256) return s.n_keys >= 2 * kTileKeys;
    return (s.head_dim == 64 || s.head_dim == 128) && s.n_keys >= kTileKeys;
}

size_t ea_mma_image_bytes(const ea_shape& s) {
    const int Gq = s.n_q_heads / s.n_kv_heads;
    const int hpc = 256 / s.head_dim;
    const size_t subsets = (size_t)((Gq + hpc - 1) / hpc);
    const size_t diag_blocks = s.head_dim <= 128 ? (size_t)hpc * (s.head_dim / 16) * 512 : 0;
    return (size_t)s.n_units * s.n_kv_heads * subsets *
           ((size_t)hpc * s.head_dim * s.head_dim * 2 + (size_t)hpc * s.head_dim * 32 + diag_blocks);
}

size_t ea_mma_vec_bytes(const ea_shape& s) {
    return (size_t)s.n_units * s.n_q_heads * s.head_dim * sizeof(float);
}

size_t ea_mma_lse_part_bytes(const ea_shape& s) {
    // at most one work unit per 128-key tile
    return (size_t)s.n_units * s.n_q_heads * (size_t)((s.n_keys + kTileKeys - 1) / kTileKeys) * 2 * sizeof(float);
}

ea_status ea_launch_logits_mma(const ea_ctx* ctx, const ea_shape& s, const __nv_bfloat16* k,
                               const ea_quad_form& form, void* image, float* vec,
                               float* logits, float* lse_part, int* n_chunks, cudaStream_t st) {
    uint8_t* img = static_cast<uint8_t*>(image);
    switch (s.head_dim) {
        case 64:
            return launch_mma<64, false, false>(ctx, s, k, form, img, vec, logits, lse_part, n_chunks, st);
        case 128:
            return launch_mma<128, false, false>(ctx, s, k, form, img, vec, logits, lse_part, n_chunks, st);
        case 256:
            return launch_mma<256, true, false>(ctx, s, k, form, img, vec, logits, lse_part, n_chunks, st);
        default:
            return EA_ERR_UNSUPPORTED;
    }
}

bool ea_mma_q8_supported(const ea_shape& s) { return ea_mma_path_supported(s); }

ea_status ea_launch_logits_mma_q8(const ea_ctx* ctx, const ea_shape& s, const uint8_t* k_q8,
                                  const ea_quad_form& form, void* image, float* vec, float* logits,
                                  float* lse_part, int* n_chunks, cudaStream_t st) {
    uint8_t* img = static_cast<uint8_t*>(image);
    switch (s.head_dim) {
        case 64:
            return launch_mma<64, false, true>(ctx, s, k_q8, form, img, vec, logits, lse_part, n_chunks, st);
        case 128:
            return launch_mma<128, false, true>(ctx, s, k_q8, form, img, vec, logits, lse_part, n_chunks, st);
        case 256:
            return launch_mma<256, true, true>(ctx, s, k_q8, form, img, vec, logits, lse_part, n_chunks, st);
        default:
            return EA_ERR_UNSUPPORTED;
    }
}
