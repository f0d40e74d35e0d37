// Eviction and compaction: per (unit, KV head) the n_kept highest scores, ties
// to the lowest index, kept indices ascending; then a row gather of K and V.
//
// select_cluster_kernel: a cluster of up to 8 CTAs per head.  Every CTA keeps its slice of the
// head's scores in shared memory (one read from HBM/L2), the radix passes run there, the per-pass
// histograms meet in the shared memory of the cluster's first CTA (distributed shared memory), and
// the ordered emission uses the slice totals exchanged the same way.  Heads too long for eight
// slices fall back to select_kernel.
// select_kernel: one CTA per head.  MSB-first radix select (4 passes of 8 bits)
// on an order-preserving integer image of the fp32 scores finds the value tau
// of the n_kept-th largest score and how many scores equal to tau are still
// needed; one ordered pass (block-wide prefix sums over consecutive chunks)
// then emits every index with score > tau and the first `need_eq` indices with
// score == tau, in ascending order.  Integer work only: bit-exact and
// reproducible.
// gather_kernel: lanes copy 16 bytes each; a warp moves 512 contiguous output
// bytes per step.
//
// Head-adaptive eviction (the head-adaptive paragraph of Sec. 2.2): every head keeps its n_floor
// best pairs and the rest of the unit's budget goes to the best remaining pairs of the unit.  The
// kept set of a head is then a prefix of that head's own order, so all that is new is the count
// m_g per head.  With c_g(x) the number of keys of head g at or above x, the pairs at or above x
// that are not safeguarded number f(x) = sum_g max(0, c_g(x) - n_floor), and the threshold T is the
// largest x with f(x) >= places.  adaptive_hist_kernel / adaptive_decide_kernel find T with the same
// MSB-first radix search, one 256-bin histogram per head and pass; the last decide step hands the
// pairs equal to T to the heads in head order and writes m_g and the offsets.  The per-head
// selection kernels then run with those counts.
#include <cooperative_groups.h>

#include "ea_internal.h"

namespace {

constexpr int kSelThreads = 1024;
constexpr int kItems = 4;

// Monotone map float -> uint32 (larger float, larger integer); -0 counts as +0.
__device__ __forceinline__ uint32_t order_key(float x) {
    uint32_t b = __float_as_uint(x);
    if (b == 0x80000000u) b = 0u;
    return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Where a head's kept indices go and how many there are: n_kept each, one head after the other, or
// (head-adaptive) a count per head and an offset per head inside the unit's range of the output.
struct HeadPlan {
    const int32_t* head_kept;     // [units * Hkv] or nullptr
    const int32_t* head_off;      // [units, Hkv + 1]
    int Hkv;
    int unit_stride;              // kept indices per unit
};

__device__ __forceinline__ int32_t* head_output(const HeadPlan& plan, int head, int32_t* kept_idx, int& n_kept) {
    if (!plan.head_kept) return kept_idx + (size_t)head * n_kept;
    const int u = head / plan.Hkv, g = head % plan.Hkv;
    n_kept = plan.head_kept[head];
    return kept_idx + (size_t)u * plan.unit_stride + plan.head_off[(size_t)u * (plan.Hkv + 1) + g];
}

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int n, int n_kept, const HeadPlan plan,
              int32_t* __restrict__ kept_idx) {
    __shared__ unsigned hist[256];
    __shared__ unsigned sh_prefix, sh_need;
    __shared__ unsigned warp_tot[32];
    __shared__ unsigned chunk_tot;

    const float* s = scores + (size_t)blockIdx.x * n;
    int32_t* out = head_output(plan, (int)blockIdx.x, kept_idx, n_kept);
    const int tid = threadIdx.x, lane = tid % 32, warp = tid / 32;
    if (n_kept <= 0) return;

    unsigned prefix = 0u, mask = 0u, need = (unsigned)n_kept;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        for (int i0 = 0; i0 < n; i0 += kSelThreads) {
            const int i = i0 + tid;
            const bool live = i < n;
            const uint32_t key = live ? order_key(s[i]) : 0u;
            const bool cand = live && ((key & mask) == prefix);
            const unsigned digit = (key >> shift) & 255u;
            const unsigned voters = __ballot_sync(0xffffffffu, cand);
            if (cand) {
                const unsigned peers = __match_any_sync(voters, digit);
                if (lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (unsigned)__popc(peers));
            }
        }
        __syncthreads();
        if (tid == 0) {
            unsigned cum = 0u, digit = 0u;
            for (int b = 255; b >= 0; --b) {
                if (cum + hist[b] >= need) { digit = (unsigned)b; break; }
                cum += hist[b];
            }
            sh_prefix = prefix | (digit << shift);
            sh_need = need - cum;
        }
        __syncthreads();
        prefix = sh_prefix;
        need = sh_need;
        mask |= 255u << shift;
    }
    const uint32_t tau = prefix;      // image of the n_kept-th largest score
    const unsigned need_eq = need;    // how many scores equal to tau are kept

    unsigned run_gt = 0u, run_eq = 0u;
    const bool vec_ok = (n % 4) == 0;
    for (int base = 0; base < n; base += kSelThreads * kItems) {
        const int i0 = base + tid * kItems;
        uint32_t key[kItems];
        if (vec_ok && i0 + kItems <= n) {
            const float4 x = *reinterpret_cast<const float4*>(s + i0);
            key[0] = order_key(x.x); key[1] = order_key(x.y);
            key[2] = order_key(x.z); key[3] = order_key(x.w);
        } else {
#pragma unroll
            for (int j = 0; j < kItems; ++j) key[j] = (i0 + j < n) ? order_key(s[i0 + j]) : 0u;
        }
        unsigned cnt = 0u;            // low 16 bits: # > tau, high 16 bits: # == tau
#pragma unroll
        for (int j = 0; j < kItems; ++j)
            if (i0 + j < n) cnt += (key[j] > tau ? 1u : 0u) + (key[j] == tau ? 0x10000u : 0u);
        // block-wide exclusive prefix sum of cnt
        unsigned incl = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned o = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            unsigned w = warp_tot[lane], wi = w;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned o = __shfl_up_sync(0xffffffffu, wi, off);
                if (lane >= off) wi += o;
            }
            warp_tot[lane] = wi - w;
            if (lane == 31) chunk_tot = wi;
        }
        __syncthreads();
        const unsigned excl = incl - cnt + warp_tot[warp];
        unsigned gt_before = run_gt + (excl & 0xffffu);
        unsigned eq_before = run_eq + (excl >> 16);
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            if (i0 + j >= n) break;
            if (key[j] > tau) {
                out[gt_before + min(eq_before, need_eq)] = i0 + j;
                ++gt_before;
            } else if (key[j] == tau) {
                if (eq_before < need_eq) out[gt_before + eq_before] = i0 + j;
                ++eq_before;
            }
        }
        run_gt += chunk_tot & 0xffffu;
        run_eq += chunk_tot >> 16;
        __syncthreads();              // warp_tot / chunk_tot are rewritten next chunk
    }
}

namespace cg = cooperative_groups;

constexpr int kClThreads = 512;
constexpr int kClMaxSlice = 49152;      // keys of one CTA's slice: 192 KiB of shared memory at most

// Cluster of C CTAs per head; CTA `rank` owns keys [rank * slice, min(n, (rank + 1) * slice)).
__global__ void __launch_bounds__(kClThreads)
select_cluster_kernel(const float* __restrict__ scores, int n, int n_kept, int slice, const HeadPlan plan,
                      int32_t* __restrict__ kept_idx) {
    extern __shared__ uint32_t keys[];                 // [slice] order keys of this CTA's slice
    __shared__ unsigned hist[256];                     // local histogram; in rank 0 also the cluster's sum
    __shared__ unsigned ghist[4][256];                 // rank 0: per pass, histogram summed over the cluster
    __shared__ unsigned slice_cnt[2][8];               // rank 0: per-slice (# > tau, # == tau)
    __shared__ unsigned warp_tot[kClThreads / 32];
    __shared__ unsigned chunk_tot;
    __shared__ unsigned sh_prefix, sh_need;

    cg::cluster_group cluster = cg::this_cluster();
    const unsigned C = cluster.num_blocks();
    const unsigned rank = cluster.block_rank();
    const int head = blockIdx.x / C;
    const int tid = threadIdx.x, lane = tid % 32, warp = tid / 32;
    const int begin = (int)rank * slice;
    const int count = max(0, min(n, begin + slice) - begin);
    const float* s = scores + (size_t)head * n + begin;
    int32_t* out = head_output(plan, head, kept_idx, n_kept);
    if (n_kept <= 0) return;                           // the same for every CTA of the cluster
    unsigned* ghist0 = cluster.map_shared_rank(&ghist[0][0], 0);
    unsigned* cnt0 = cluster.map_shared_rank(&slice_cnt[0][0], 0);

    // slice -> shared memory as order-preserving integers
    const bool vec_ok = ((((size_t)head * n + begin) & 3) == 0);
    if (vec_ok) {
        for (int i = tid * 4; i < count; i += kClThreads * 4) {
            if (i + 4 <= count) {
                const float4 x = *reinterpret_cast<const float4*>(s + i);
                keys[i] = order_key(x.x); keys[i + 1] = order_key(x.y);
                keys[i + 2] = order_key(x.z); keys[i + 3] = order_key(x.w);
            } else {
                for (int j = i; j < count; ++j) keys[j] = order_key(s[j]);
            }
        }
    } else {
        for (int i = tid; i < count; i += kClThreads) keys[i] = order_key(s[i]);
    }
    for (int i = tid; i < 4 * 256; i += kClThreads) (&ghist[0][0])[i] = 0u;
    cluster.sync();

    unsigned prefix = 0u, mask = 0u, need = (unsigned)n_kept;
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        for (int i0 = 0; i0 < count; i0 += kClThreads) {
            const int i = i0 + tid;
            const bool live = i < count;
            const uint32_t key = live ? keys[i] : 0u;
            const bool cand = live && ((key & mask) == prefix);
            const unsigned digit = (key >> shift) & 255u;
            const unsigned voters = __ballot_sync(0xffffffffu, cand);
            if (cand) {
                const unsigned peers = __match_any_sync(voters, digit);
                if (lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (unsigned)__popc(peers));
            }
        }
        __syncthreads();
        if (tid < 256 && hist[tid]) atomicAdd(&ghist0[pass * 256 + tid], hist[tid]);   // integer sums: order-free
        cluster.sync();
        // every CTA fetches the cluster's histogram once (256 parallel remote reads), then warp 0
        // finds the digit where the count from the top reaches `need`: lane l owns bins 8l .. 8l+7
        if (tid < 256) hist[tid] = ghist0[pass * 256 + tid];
        __syncthreads();
        if (warp == 0) {
            unsigned b8[8], mine = 0u;
#pragma unroll
            for (int j = 0; j < 8; ++j) { b8[j] = hist[8 * lane + j]; mine += b8[j]; }
            unsigned above = mine;            // inclusive suffix sum over lanes lane .. 31
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned o = __shfl_down_sync(0xffffffffu, above, off);
                if (lane + off < 32) above += o;
            }
            const unsigned cum_hi = above - mine;             // bins above this lane's eight
            const bool here = cum_hi < need && above >= need; // the threshold digit is one of mine
            if (here) {
                unsigned cum = cum_hi, digit = 0u;
#pragma unroll
                for (int j = 7; j >= 0; --j) {
                    if (cum + b8[j] >= need) { digit = (unsigned)(8 * lane + j); break; }
                    cum += b8[j];
                }
                sh_prefix = prefix | (digit << shift);
                sh_need = need - cum;
            }
        }
        __syncthreads();
        prefix = sh_prefix;
        need = sh_need;
        mask |= 255u << shift;
    }
    const uint32_t tau = prefix;        // image of the n_kept-th largest score
    const unsigned need_eq = need;      // how many scores equal to tau are kept, lowest indices first

    // slice totals, then this slice's offsets
    unsigned my_gt = 0u, my_eq = 0u;
    for (int i = tid; i < count; i += kClThreads) {
        const uint32_t key = keys[i];
        my_gt += key > tau ? 1u : 0u;
        my_eq += key == tau ? 1u : 0u;
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        my_gt += __shfl_xor_sync(0xffffffffu, my_gt, off);
        my_eq += __shfl_xor_sync(0xffffffffu, my_eq, off);
    }
    if (lane == 0) warp_tot[warp] = my_gt | (my_eq << 16);     // a slice holds fewer than 65536 keys
    __syncthreads();
    if (tid == 0) {
        unsigned g = 0u, e = 0u;
        for (int w = 0; w < kClThreads / 32; ++w) { g += warp_tot[w] & 0xffffu; e += warp_tot[w] >> 16; }
        cnt0[rank] = g;
        cnt0[8 + rank] = e;
    }
    cluster.sync();
    unsigned run_gt = 0u, run_eq = 0u;
    for (unsigned r = 0; r < rank; ++r) { run_gt += cnt0[r]; run_eq += cnt0[8 + r]; }
    __syncthreads();

    // ordered emission of this slice (block-wide prefix sums over consecutive chunks)
    for (int base = 0; base < count; base += kClThreads * kItems) {
        const int i0 = base + tid * kItems;
        uint32_t key[kItems];
#pragma unroll
        for (int j = 0; j < kItems; ++j) key[j] = (i0 + j < count) ? keys[i0 + j] : 0u;
        unsigned cnt = 0u;            // low 16 bits: # > tau, high 16 bits: # == tau
#pragma unroll
        for (int j = 0; j < kItems; ++j)
            if (i0 + j < count) cnt += (key[j] > tau ? 1u : 0u) + (key[j] == tau ? 0x10000u : 0u);
        unsigned incl = cnt;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const unsigned o = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += o;
        }
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            unsigned w = lane < kClThreads / 32 ? warp_tot[lane] : 0u, wi = w;
#pragma unroll
            for (int off = 1; off < 32; off <<= 1) {
                const unsigned o = __shfl_up_sync(0xffffffffu, wi, off);
                if (lane >= off) wi += o;
            }
            if (lane < kClThreads / 32) warp_tot[lane] = wi - w;
            if (lane == 31) chunk_tot = wi;
        }
        __syncthreads();
        const unsigned excl = incl - cnt + warp_tot[warp];
        unsigned gt_before = run_gt + (excl & 0xffffu);
        unsigned eq_before = run_eq + (excl >> 16);
#pragma unroll
        for (int j = 0; j < kItems; ++j) {
            if (i0 + j >= count) break;
            if (key[j] > tau) {
                out[gt_before + min(eq_before, need_eq)] = begin + i0 + j;
                ++gt_before;
            } else if (key[j] == tau) {
                if (eq_before < need_eq) out[gt_before + eq_before] = begin + i0 + j;
                ++eq_before;
            }
        }
        run_gt += chunk_tot & 0xffffu;
        run_eq += chunk_tot >> 16;
        __syncthreads();
    }
    cluster.sync();       // rank 0's shared memory stays alive until every CTA has read it
}

template <int D>
__global__ void gather_kernel(const int32_t* __restrict__ kept_idx, long long n_rows_out, int n,   // n: rows per head in k, v
                              int n_kept, const uint4* __restrict__ k, const uint4* __restrict__ v,
                              uint4* __restrict__ k_out, uint4* __restrict__ v_out) {
    constexpr int LPR = D / 8;                 // 16-byte pieces per row
    const long long total = n_rows_out * LPR;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        const long long row = t / LPR;
        const int piece = (int)(t % LPR);
        const long long head = row / n_kept;
        const long long src = head * n + kept_idx[row];
        k_out[t] = __ldg(k + src * LPR + piece);
        v_out[t] = __ldg(v + src * LPR + piece);
    }
}


// ------------------------------------------------------------------------------------------
// Head-adaptive counts.
constexpr int kAdSpan = 16384;        // keys per CTA of the histogram kernel

struct AdaptiveWs {
    unsigned* ghist;      // [4][heads][256]
    unsigned* prefix;     // [units]  digits of the threshold found so far
    unsigned* above;      // [heads]  keys of the head above every key that shares the prefix
    int32_t* head_kept;   // [heads]  m_g
};

__host__ __device__ inline AdaptiveWs adaptive_ws(void* ws, size_t units, size_t heads) {
    AdaptiveWs a;
    a.ghist = static_cast<unsigned*>(ws);
    a.prefix = a.ghist + 4 * heads * 256;
    a.above = a.prefix + units;
    a.head_kept = reinterpret_cast<int32_t*>(a.above + heads);
    return a;
}

// Histogram of digit `pass` (MSB first) over the keys of a head that share the unit's prefix.
__global__ void __launch_bounds__(kSelThreads)
adaptive_hist_kernel(const float* __restrict__ scores, int n, int Hkv, int pass,
                     const unsigned* __restrict__ prefix_u, unsigned* __restrict__ ghist_pass) {
    __shared__ unsigned hist[256];
    const int head = blockIdx.x;
    const int tid = threadIdx.x, lane = tid % 32;
    const int shift = 24 - 8 * pass;
    const unsigned mask = pass == 0 ? 0u : 0xffffffffu << (32 - 8 * pass);
    const unsigned prefix = pass == 0 ? 0u : prefix_u[head / Hkv];
    const float* s = scores + (size_t)head * n;
    if (tid < 256) hist[tid] = 0u;
    __syncthreads();
    const int begin = blockIdx.y * kAdSpan, end = min(n, begin + kAdSpan);
    for (int i0 = begin; i0 < end; i0 += kSelThreads) {
        const int i = i0 + tid;
        const bool live = i < end;
        const uint32_t key = live ? order_key(s[i]) : 0u;
        const bool cand = live && ((key & mask) == prefix);
        const unsigned digit = (key >> shift) & 255u;
        const unsigned voters = __ballot_sync(0xffffffffu, cand);
        if (cand) {
            const unsigned peers = __match_any_sync(voters, digit);
            if (lane == __ffs(peers) - 1) atomicAdd(&hist[digit], (unsigned)__popc(peers));
        }
    }
    __syncthreads();
    if (tid < 256 && hist[tid]) atomicAdd(&ghist_pass[(size_t)head * 256 + tid], hist[tid]);   // integer sums: order-free
}

// Inclusive suffix sum over the 256 threads of a block (thread b gets the sum over threads >= b).
__device__ __forceinline__ unsigned block_suffix_sum(unsigned v, unsigned* warp_tot) {
    const int lane = threadIdx.x % 32, warp = threadIdx.x / 32;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const unsigned o = __shfl_down_sync(0xffffffffu, v, off);
        if (lane + off < 32) v += o;
    }
    __syncthreads();                       // warp_tot may still be read from the previous call
    if (lane == 0) warp_tot[warp] = v;
    __syncthreads();
    for (int w = warp + 1; w < 8; ++w) v += warp_tot[w];
    return v;
}

// One CTA of 256 threads (one per bin) per unit: the digit of the threshold at this pass; after the
// last pass also the count of every head and the offsets.
__global__ void __launch_bounds__(256)
adaptive_decide_kernel(int Hkv, int n_floor, unsigned long long places, int pass,
                       const unsigned* __restrict__ ghist_pass, unsigned* __restrict__ prefix_u,
                       unsigned* __restrict__ above, int32_t* __restrict__ head_kept,
                       int32_t* __restrict__ head_off) {
    __shared__ unsigned warp_tot[8];
    __shared__ int sh_digit;
    const int u = blockIdx.x, b = threadIdx.x;
    const int shift = 24 - 8 * pass;
    // f(b): pairs of the unit, outside the safeguard shares, whose key is at or above bin b of the prefix
    unsigned long long f = 0ull;
    for (int g = 0; g < Hkv; ++g) {
        const size_t head = (size_t)u * Hkv + g;
        const unsigned at_or_above = above[head] + block_suffix_sum(ghist_pass[head * 256 + b], warp_tot);
        f += at_or_above > (unsigned)n_floor ? at_or_above - (unsigned)n_floor : 0u;
    }
    if (b == 0) sh_digit = 0;
    __syncthreads();
    if (f >= places) atomicMax(&sh_digit, b);          // f falls as b rises: the largest bin that still reaches `places`
    __syncthreads();
    const int digit = sh_digit;
    // keys above the chosen bin are above the threshold for good
    for (int g = 0; g < Hkv; ++g) {
        const size_t head = (size_t)u * Hkv + g;
        const unsigned h = ghist_pass[head * 256 + b];
        const unsigned higher = block_suffix_sum(b > digit ? h : 0u, warp_tot);
        if (b == 0) above[head] += higher;
    }
    if (b == 0) prefix_u[u] |= (unsigned)digit << shift;
    if (pass < 3) return;
    __syncthreads();
    if (b == 0) {
        // threshold T = prefix: every pair above T outside the safeguard shares is kept, the pairs equal
        // to T fill what is left, heads in order (inside a head: lowest index first)
        unsigned long long taken_above = 0ull;
        for (int g = 0; g < Hkv; ++g) {
            const unsigned gt = above[(size_t)u * Hkv + g];
            taken_above += gt > (unsigned)n_floor ? gt - (unsigned)n_floor : 0u;
        }
        unsigned long long left = places - taken_above;
        int32_t off = 0;
        for (int g = 0; g < Hkv; ++g) {
            const size_t head = (size_t)u * Hkv + g;
            const unsigned gt = above[head], eq = ghist_pass[head * 256 + digit];
            const unsigned base = gt > (unsigned)n_floor ? gt : (unsigned)n_floor;
            const unsigned free_eq = gt + eq > base ? gt + eq - base : 0u;
            const unsigned take = (unsigned long long)free_eq < left ? free_eq : (unsigned)left;
            left -= take;
            head_kept[head] = (int32_t)(base + take);
            head_off[(size_t)u * (Hkv + 1) + g] = off;
            off += (int32_t)(base + take);
        }
        head_off[(size_t)u * (Hkv + 1) + Hkv] = off;
    }
}

template <int D>
__global__ void gather_adaptive_kernel(const int32_t* __restrict__ kept_idx, const int32_t* __restrict__ head_off,
                                       long long n_rows_out, int n, int Hkv, int unit_stride,
                                       const uint4* __restrict__ k, const uint4* __restrict__ v,
                                       uint4* __restrict__ k_out, uint4* __restrict__ v_out) {
    constexpr int LPR = D / 8;                 // 16-byte pieces per row
    const long long total = n_rows_out * LPR;
    const long long stride = (long long)gridDim.x * blockDim.x;
    for (long long t = (long long)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += stride) {
        const long long row = t / LPR;
        const int piece = (int)(t % LPR);
        const long long u = row / unit_stride;
        const int j = (int)(row % unit_stride);
        // the head whose range holds j: the last g with head_off[g] <= j
        const int32_t* off = head_off + u * (Hkv + 1);
        int lo = 0, hi = Hkv - 1;
        while (lo < hi) {
            const int mid = (lo + hi + 1) / 2;
            if (off[mid] <= j) lo = mid;
            else hi = mid - 1;
        }
        const long long src = (u * Hkv + lo) * n + kept_idx[row];
        k_out[t] = __ldg(k + src * LPR + piece);
        v_out[t] = __ldg(v + src * LPR + piece);
    }
}

// In-place compaction of one head of one tensor per CTA: row j of the head receives row idx[j].
// idx is ascending, so idx[j] >= j: rows only move towards the front.  The CTA walks the kept rows
// in chunks, front to back; all of a chunk's source rows are in registers before any of its
// destination rows is written (the barrier), and a later chunk only reads rows at or behind its own
// first destination row, which earlier chunks never write.
constexpr int kIpThreads = 256;
constexpr int kIpLoads = 4;            // 16-byte pieces per thread and chunk

template <int D>
__global__ void __launch_bounds__(kIpThreads)
compact_inplace_kernel(const int32_t* __restrict__ kept_idx, int n, int n_kept, uint4* k, uint4* v) {
    constexpr int LPR = D / 8;                                  // 16-byte pieces per row
    constexpr int kChunkRows = kIpThreads * kIpLoads / LPR;
    const long long head = blockIdx.x;
    uint4* rows = (blockIdx.y == 0 ? k : v) + head * (long long)n * LPR;
    const int32_t* idx = kept_idx + head * (long long)n_kept;
    for (int j0 = 0; j0 < n_kept; j0 += kChunkRows) {
        uint4 x[kIpLoads];
        int src[kIpLoads];
#pragma unroll
        for (int i = 0; i < kIpLoads; ++i) {
            const int t = i * kIpThreads + threadIdx.x;
            const int j = j0 + t / LPR;
            src[i] = j < n_kept ? idx[j] : -1;
            if (src[i] >= 0 && src[i] != j) x[i] = rows[(long long)src[i] * LPR + t % LPR];
        }
        __syncthreads();
#pragma unroll
        for (int i = 0; i < kIpLoads; ++i) {
            const int t = i * kIpThreads + threadIdx.x;
            const int j = j0 + t / LPR;
            if (src[i] >= 0 && src[i] != j) rows[(long long)j * LPR + t % LPR] = x[i];
        }
    }
}

// Unordered in-place compaction of one head of one tensor per CTA.  `sel` holds the head's kept positions
// ascending.  Kept rows below n_kept stay; the kept rows at or beyond n_kept (the tail of `sel`) move, in
// order, into the evicted positions below n_kept, in order.  Sources lie at or beyond n_kept and
// destinations below it, so no move can disturb another.  where[j] = the original row now at j.
constexpr int kFillThreads = 256;

template <int D>
__global__ void __launch_bounds__(kFillThreads)
compact_fill_kernel(const int32_t* __restrict__ sel, int cap, int n_kept, int32_t* __restrict__ where, uint4* k,
                    uint4* v) {
    constexpr int LPR = D / 8;                         // 16-byte pieces per row
    extern __shared__ int32_t fill_smem[];             // [n_kept] kept positions, then [n_kept] destinations of the movers
    int32_t* a = fill_smem;
    int32_t* dst_of = fill_smem + n_kept;
    __shared__ int m_sh;
    const long long head = blockIdx.x;
    const int32_t* src_idx = sel + head * (long long)n_kept;
    for (int j = threadIdx.x; j < n_kept; j += kFillThreads) a[j] = src_idx[j];
    __syncthreads();
    if (threadIdx.x == 0) {
        int lo = 0, hi = n_kept;                       // first j with a[j] >= n_kept: the rows before it stay
        while (lo < hi) {
            const int mid = (lo + hi) / 2;
            if (a[mid] < n_kept) lo = mid + 1;
            else hi = mid;
        }
        m_sh = lo;
    }
    __syncthreads();
    const int m = m_sh;
    for (int p = threadIdx.x; p < n_kept; p += kFillThreads) {
        int lo = 0, hi = m;                            // kept positions below p
        while (lo < hi) {
            const int mid = (lo + hi) / 2;
            if (a[mid] < p) lo = mid + 1;
            else hi = mid;
        }
        const bool stays = lo < m && a[lo] == p;
        int32_t w = p;
        if (!stays) {
            const int r = p - lo;                      // rank of this hole = rank of the mover that fills it
            w = a[m + r];
            dst_of[r] = p;
        }
        if (blockIdx.y == 0) where[head * (long long)n_kept + p] = w;
    }
    __syncthreads();
    uint4* rows = (blockIdx.y == 0 ? k : v) + head * (long long)cap * LPR;
    const int n_moves = n_kept - m;
    for (int t = threadIdx.x; t < n_moves * LPR; t += kFillThreads) {
        const int r = t / LPR, piece = t % LPR;
        rows[(long long)dst_of[r] * LPR + piece] = rows[(long long)a[m + r] * LPR + piece];
    }
}

// A per-token fp32 array of a head follows its rows through an in-place compaction: position j receives the
// value of row idx[j] >= j (ascending kept positions, or the original row now at j after the unordered form,
// where movers come from beyond n_kept).  One CTA per head walks the positions in chunks, a chunk's sources
// in registers before its destinations are written; a later chunk reads at or behind its own first
// destination, which earlier chunks never write.
constexpr int kCarryThreads = 256;
__global__ void __launch_bounds__(kCarryThreads)
carry_f32_kernel(const int32_t* __restrict__ idx_all, int cap, int n_kept, float* values) {
    const long long head = blockIdx.x;
    float* vs = values + head * (long long)cap;
    const int32_t* idx = idx_all + head * (long long)n_kept;
    for (int j0 = 0; j0 < n_kept; j0 += kCarryThreads) {
        const int j = j0 + threadIdx.x;
        const int src = j < n_kept ? idx[j] : -1;
        const float x = src >= 0 ? vs[src] : 0.f;
        __syncthreads();
        if (src >= 0) vs[j] = x;
    }
}

}  // namespace

ea_status ea_launch_carry_f32(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* idx, float* values,
                              cudaStream_t st) {
    if (n_kept <= 0) return EA_OK;
    carry_f32_kernel<<<(unsigned)(s.n_units * s.n_kv_heads), kCarryThreads, 0, st>>>(idx, ea_kv_cap(s), n_kept, values);
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}

static ea_status launch_select(const ea_ctx* ctx, const ea_shape& s, const float* scores, int n_kept,
                               const HeadPlan& plan, int32_t* kept_idx, cudaStream_t st) {
    if (n_kept <= 0) return EA_OK;
    ea_count_launches(ctx, 1);
    const int heads = s.n_units * s.n_kv_heads;
    // slices of about 16 K keys, at most 8 CTAs per head (the portable cluster size)
    int C = 1;
    while (C < 8 && (s.n_keys + C - 1) / C > 16384) C *= 2;
    int slice = ((s.n_keys + C - 1) / C + 3) / 4 * 4;
    if (slice <= kClMaxSlice && (long long)heads * C < 0x7fffffffLL) {
        const size_t smem = (size_t)slice * sizeof(uint32_t);
        if (cudaFuncSetAttribute(select_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) !=
            cudaSuccess)
            return EA_ERR_CUDA;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(heads * C));
        cfg.blockDim = dim3(kClThreads);
        cfg.dynamicSmemBytes = smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)C;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelEx(&cfg, select_cluster_kernel, scores, s.n_keys, n_kept, slice, plan, kept_idx) !=
            cudaSuccess)
            return EA_ERR_CUDA;
    } else {
        select_kernel<<<heads, kSelThreads, 0, st>>>(scores, s.n_keys, n_kept, plan, kept_idx);
    }
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_select(const ea_ctx* ctx, const ea_shape& s, const float* scores, int n_kept,
                           int32_t* kept_idx, cudaStream_t st) {
    const HeadPlan plan = {nullptr, nullptr, s.n_kv_heads, 0};
    return launch_select(ctx, s, scores, n_kept, plan, kept_idx, st);
}

size_t ea_adaptive_ws_bytes(const ea_shape& s) {
    const size_t units = (size_t)s.n_units, heads = units * (size_t)s.n_kv_heads;
    return (4 * heads * 256 + units + 2 * heads) * sizeof(unsigned);
}

ea_status ea_launch_select_adaptive(const ea_ctx* ctx, const ea_shape& s, const float* scores, int n_kept,
                                    int n_floor, void* ws, int32_t* kept_idx, int32_t* head_offsets,
                                    cudaStream_t st) {
    const size_t units = (size_t)s.n_units, heads = units * (size_t)s.n_kv_heads;
    const AdaptiveWs a = adaptive_ws(ws, units, heads);
    EA_CUDA_TRY(cudaMemsetAsync(ws, 0, ea_adaptive_ws_bytes(s), st));
    const unsigned long long places = (unsigned long long)s.n_kv_heads * (unsigned long long)(n_kept - n_floor);
    const dim3 hist_grid((unsigned)heads, (unsigned)((s.n_keys + kAdSpan - 1) / kAdSpan));
    if (hist_grid.y > 65535u) return EA_ERR_UNSUPPORTED;
    for (int pass = 0; pass < 4; ++pass) {
        unsigned* gh = a.ghist + (size_t)pass * heads * 256;
        if (s.n_keys > 0)
            adaptive_hist_kernel<<<hist_grid, kSelThreads, 0, st>>>(scores, s.n_keys, s.n_kv_heads, pass, a.prefix, gh);
        adaptive_decide_kernel<<<(unsigned)units, 256, 0, st>>>(s.n_kv_heads, n_floor, places, pass, gh, a.prefix,
                                                                a.above, a.head_kept, head_offsets);
        ea_count_launches(ctx, s.n_keys > 0 ? 2 : 1);
    }
    if (EA_CHECK_LAUNCH() != EA_OK) return EA_ERR_CUDA;
    const HeadPlan plan = {a.head_kept, head_offsets, s.n_kv_heads, s.n_kv_heads * n_kept};
    // n_kept here only says "some head may keep something"; every head reads its own count
    return launch_select(ctx, s, scores, n_kept, plan, kept_idx, st);
}

ea_status ea_launch_gather_adaptive(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* kept_idx,
                                    const int32_t* head_offsets, const __nv_bfloat16* k, const __nv_bfloat16* v,
                                    __nv_bfloat16* k_out, __nv_bfloat16* v_out, cudaStream_t st) {
    if (n_kept <= 0) return EA_OK;
    ea_count_launches(ctx, 1);
    const int unit_stride = s.n_kv_heads * n_kept;
    const long long rows = (long long)s.n_units * unit_stride;
    const int threads = 256;
    const long long pieces = rows * (s.head_dim / 8);
    long long want = (pieces + threads - 1) / threads;
    const long long cap = (long long)ctx->sm_count * 16;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    const uint4* k4 = reinterpret_cast<const uint4*>(k);
    const uint4* v4 = reinterpret_cast<const uint4*>(v);
    uint4* ko = reinterpret_cast<uint4*>(k_out);
    uint4* vo = reinterpret_cast<uint4*>(v_out);
    switch (s.head_dim) {
        case 64:
            gather_adaptive_kernel<64><<<grid, threads, 0, st>>>(kept_idx, head_offsets, rows, ea_kv_cap(s), s.n_kv_heads,
                                                                 unit_stride, k4, v4, ko, vo);
            break;
        case 128:
            gather_adaptive_kernel<128><<<grid, threads, 0, st>>>(kept_idx, head_offsets, rows, ea_kv_cap(s), s.n_kv_heads,
                                                                  unit_stride, k4, v4, ko, vo);
            break;
        case 256:
            gather_adaptive_kernel<256><<<grid, threads, 0, st>>>(kept_idx, head_offsets, rows, ea_kv_cap(s), s.n_kv_heads,
                                                                  unit_stride, k4, v4, ko, vo);
            break;
        default:
            return EA_ERR_UNSUPPORTED;
    }
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_gather(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* kept_idx,
                           const __nv_bfloat16* k, const __nv_bfloat16* v, __nv_bfloat16* k_out,
                           __nv_bfloat16* v_out, cudaStream_t st) {
    if (n_kept <= 0) return EA_OK;
    ea_count_launches(ctx, 1);
    const long long rows = (long long)s.n_units * s.n_kv_heads * n_kept;
    const int threads = 256;
    const long long pieces = rows * (s.head_dim / 8);
    long long want = (pieces + threads - 1) / threads;
    const long long cap = (long long)ctx->sm_count * 16;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    const uint4* k4 = reinterpret_cast<const uint4*>(k);
    const uint4* v4 = reinterpret_cast<const uint4*>(v);
    uint4* ko = reinterpret_cast<uint4*>(k_out);
    uint4* vo = reinterpret_cast<uint4*>(v_out);
    switch (s.head_dim) {
        case 64:
            gather_kernel<64><<<grid, threads, 0, st>>>(kept_idx, rows, ea_kv_cap(s), n_kept, k4, v4, ko, vo);
            break;
        case 128:
            gather_kernel<128><<<grid, threads, 0, st>>>(kept_idx, rows, ea_kv_cap(s), n_kept, k4, v4, ko, vo);
            break;
        case 256:
            gather_kernel<256><<<grid, threads, 0, st>>>(kept_idx, rows, ea_kv_cap(s), n_kept, k4, v4, ko, vo);
            break;
        default:
            return EA_ERR_UNSUPPORTED;
    }
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_compact_inplace(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* kept_idx,
                                    void* k, void* v, cudaStream_t st, bool codes) {
    if (n_kept <= 0) return EA_OK;
    ea_count_launches(ctx, 1);
    const dim3 grid((unsigned)(s.n_units * s.n_kv_heads), 2);
    uint4* k4 = reinterpret_cast<uint4*>(k);
    uint4* v4 = reinterpret_cast<uint4*>(v);
    // the kernels count rows in 16-byte pieces of bf16: a row of d one-byte codes is a bf16 row of d / 2
    switch (codes ? s.head_dim / 2 : s.head_dim) {
        case 32: compact_inplace_kernel<32><<<grid, kIpThreads, 0, st>>>(kept_idx, ea_kv_cap(s), n_kept, k4, v4); break;
        case 64: compact_inplace_kernel<64><<<grid, kIpThreads, 0, st>>>(kept_idx, ea_kv_cap(s), n_kept, k4, v4); break;
        case 128: compact_inplace_kernel<128><<<grid, kIpThreads, 0, st>>>(kept_idx, ea_kv_cap(s), n_kept, k4, v4); break;
        case 256: compact_inplace_kernel<256><<<grid, kIpThreads, 0, st>>>(kept_idx, ea_kv_cap(s), n_kept, k4, v4); break;
        default: return EA_ERR_UNSUPPORTED;
    }
    return EA_CHECK_LAUNCH();
}

ea_status ea_launch_compact_fill(const ea_ctx* ctx, const ea_shape& s, int n_kept, const int32_t* sel,
                                 int32_t* where, void* k, void* v, cudaStream_t st, bool codes) {
    if (n_kept <= 0) return EA_OK;
    const size_t smem = 2 * (size_t)n_kept * sizeof(int32_t);
    if (smem > 200 * 1024) return EA_ERR_UNSUPPORTED;
    const dim3 grid((unsigned)(s.n_units * s.n_kv_heads), 2);
    uint4* k4 = reinterpret_cast<uint4*>(k);
    uint4* v4 = reinterpret_cast<uint4*>(v);
    const int cap = ea_kv_cap(s);
    switch (codes ? s.head_dim / 2 : s.head_dim) {
        case 32:
            EA_CUDA_TRY(cudaFuncSetAttribute(compact_fill_kernel<32>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            compact_fill_kernel<32><<<grid, kFillThreads, smem, st>>>(sel, cap, n_kept, where, k4, v4);
            break;
        case 64:
            EA_CUDA_TRY(cudaFuncSetAttribute(compact_fill_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            compact_fill_kernel<64><<<grid, kFillThreads, smem, st>>>(sel, cap, n_kept, where, k4, v4);
            break;
        case 128:
            EA_CUDA_TRY(cudaFuncSetAttribute(compact_fill_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            compact_fill_kernel<128><<<grid, kFillThreads, smem, st>>>(sel, cap, n_kept, where, k4, v4);
            break;
        case 256:
            EA_CUDA_TRY(cudaFuncSetAttribute(compact_fill_kernel<256>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
            compact_fill_kernel<256><<<grid, kFillThreads, smem, st>>>(sel, cap, n_kept, where, k4, v4);
            break;
        default:
            return EA_ERR_UNSUPPORTED;
    }
    ea_count_launches(ctx, 1);
    return EA_CHECK_LAUNCH();
}
