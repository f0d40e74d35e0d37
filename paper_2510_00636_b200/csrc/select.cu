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

__global__ void __launch_bounds__(kSelThreads)
select_kernel(const float* __restrict__ scores, int n, int n_kept, int32_t* __restrict__ kept_idx) {
    __shared__ unsigned hist[256];
    __shared__ unsigned sh_prefix, sh_need;
    __shared__ unsigned warp_tot[32];
    __shared__ unsigned chunk_tot;

    const float* s = scores + (size_t)blockIdx.x * n;
    int32_t* out = kept_idx + (size_t)blockIdx.x * n_kept;
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
select_cluster_kernel(const float* __restrict__ scores, int n, int n_kept, int slice,
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
    int32_t* out = kept_idx + (size_t)head * n_kept;
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
__global__ void gather_kernel(const int32_t* __restrict__ kept_idx, long long n_rows_out, int n,
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

}  // namespace

ea_status ea_launch_select(const ea_ctx* ctx, const ea_shape& s, const float* scores, int n_kept,
                           int32_t* kept_idx, cudaStream_t st) {
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
        if (cudaLaunchKernelEx(&cfg, select_cluster_kernel, scores, s.n_keys, n_kept, slice, kept_idx) != cudaSuccess)
            return EA_ERR_CUDA;
    } else {
        select_kernel<<<heads, kSelThreads, 0, st>>>(scores, s.n_keys, n_kept, kept_idx);
    }
    return cudaGetLastError() == cudaSuccess ? EA_OK : EA_ERR_CUDA;
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
            gather_kernel<64><<<grid, threads, 0, st>>>(kept_idx, rows, s.n_keys, n_kept, k4, v4, ko, vo);
            break;
        case 128:
            gather_kernel<128><<<grid, threads, 0, st>>>(kept_idx, rows, s.n_keys, n_kept, k4, v4, ko, vo);
            break;
        case 256:
            gather_kernel<256><<<grid, threads, 0, st>>>(kept_idx, rows, s.n_keys, n_kept, k4, v4, ko, vo);
            break;
        default:
            return EA_ERR_UNSUPPORTED;
    }
    return cudaGetLastError() == cudaSuccess ? EA_OK : EA_ERR_CUDA;
}
