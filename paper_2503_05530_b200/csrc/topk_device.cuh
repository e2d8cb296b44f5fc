// Device helpers for selection: order-preserving float keys, warp-wide bitonic
// sort in registers, block-wide bitonic sort in shared memory.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace prox {

typedef unsigned long long u64;

// float -> uint32 such that a < b  <=>  f2o(a) < f2o(b)  (finite values and infinities).
__device__ __forceinline__ uint32_t f2o(float f) {
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float o2f(uint32_t o) {
    uint32_t u = (o & 0x80000000u) ? (o & 0x7fffffffu) : ~o;
    return __uint_as_float(u);
}
// (score, row) packed so that a larger key is a better candidate; 0 is below every real entry.
__device__ __forceinline__ u64 pack_entry(float score, int32_t row) {
    return ((u64)f2o(score) << 32) | (uint32_t)row;
}
__device__ __forceinline__ float entry_score(u64 e) { return o2f((uint32_t)(e >> 32)); }
__device__ __forceinline__ int32_t entry_row(u64 e) { return (int32_t)(uint32_t)e; }

// One digit of a radix select, for one whole warp: the 256 bins of hist are walked from the top
// (descending) or from the bottom until the bin that holds the rem-th entry (rem >= 1); returns
// that bin and leaves in rem the rank inside it.  If all bins together hold fewer than rem entries
// the walk ends at its last bin, with the counts of all others taken off rem.  Lane l sums the
// eight bins 8 l .. 8 l + 7 of the walk; a prefix sum over the lanes finds the lane of the answer.
__device__ __forceinline__ int radix_digit_walk(const unsigned *hist, int &rem, bool descending) {
    const int lane = threadIdx.x & 31;
    int c[8], tot = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        const int w = 8 * lane + j;
        c[j] = (int)hist[descending ? 255 - w : w];
        tot += c[j];
    }
    int incl = tot;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, m);
        if (lane >= m) incl += y;
    }
    const unsigned reach = __ballot_sync(0xffffffffu, incl >= rem);
    const int owner = reach ? __ffs(reach) - 1 : 31;
    int r = rem - (incl - tot), j = 0;
    while (j < 7 && c[j] < r) { r -= c[j]; ++j; }
    const int w = 8 * owner + __shfl_sync(0xffffffffu, j, owner);
    rem = __shfl_sync(0xffffffffu, r, owner);
    return descending ? 255 - w : w;
}

__device__ __forceinline__ u64 shfl_xor_u64(u64 v, int m) {
    uint32_t lo = __shfl_xor_sync(0xffffffffu, (uint32_t)v, m);
    uint32_t hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(v >> 32), m);
    return ((u64)hi << 32) | lo;
}

// One compare-exchange pass of the bitonic network between the register slots it and it ^ DJ of
// every lane (keys 32 * DJ apart); k is the size of the bitonic blocks being merged.
template <int ITEMS, int DJ>
__device__ __forceinline__ void sort_pass_regs(u64 (&v)[ITEMS], int k, int lane) {
#pragma unroll
    for (int it = 0; it < ITEMS; ++it) {
        const int partner = it ^ DJ;
        if (partner > it) {
            const int e = it * 32 + lane;
            const bool desc = ((e & k) == 0);
            const u64 a = v[it], b = v[partner];
            const bool swap = desc ? (a < b) : (a > b);
            v[it] = swap ? b : a;
            v[partner] = swap ? a : b;
        }
    }
}

// Sorts ITEMS*32 keys held by one warp, DESCENDING.  Element e lives in
// v[e / 32] of lane e % 32, so after the sort v[0] of lane 0 is the largest key,
// v[0] of lane 1 the next, ... v[1] of lane 0 the 33rd, and so on.
// The passes of the network run in rolled loops (only the register slots are unrolled): the
// sort is rare next to the code that calls it, and a fully unrolled network is tens of
// kilobytes of instructions that would push that code out of the instruction cache.
template <int ITEMS>
__device__ __forceinline__ void warp_sort_desc(u64 (&v)[ITEMS]) {
    constexpr int LOG = (ITEMS == 1 ? 5 : ITEMS == 2 ? 6 : ITEMS == 4 ? 7 : ITEMS == 8 ? 8 : ITEMS == 16 ? 9 : 10);
    static_assert((32 << (LOG - 5)) == ITEMS * 32, "ITEMS must be a power of two up to 32");
    const int lane = threadIdx.x & 31;
#pragma unroll 1
    for (int lk = 1; lk <= LOG; ++lk) {
        const int k = 1 << lk;
#pragma unroll 1
        for (int lj = lk - 1; lj >= 0; --lj) {
            const int j = 1 << lj;
            if (j >= 32) {
                switch (j >> 5) {
                    case 1: if constexpr (ITEMS >= 2) sort_pass_regs<ITEMS, 1>(v, k, lane); break;
                    case 2: if constexpr (ITEMS >= 4) sort_pass_regs<ITEMS, 2>(v, k, lane); break;
                    case 4: if constexpr (ITEMS >= 8) sort_pass_regs<ITEMS, 4>(v, k, lane); break;
                    case 8: if constexpr (ITEMS >= 16) sort_pass_regs<ITEMS, 8>(v, k, lane); break;
                    default: if constexpr (ITEMS >= 32) sort_pass_regs<ITEMS, 16>(v, k, lane); break;
                }
            } else {
                const bool lower = ((lane & j) == 0);           // this lane holds the lower index of the pair
#pragma unroll
                for (int it = 0; it < ITEMS; ++it) {
                    const int e = it * 32 + lane;
                    const bool desc = ((e & k) == 0);
                    const u64 mine = v[it];
                    const u64 other = shfl_xor_u64(mine, j);
                    // descending block: lower index keeps the max; ascending block: lower keeps the min
                    const bool keep_max = (desc == lower);
                    v[it] = keep_max ? (mine > other ? mine : other) : (mine < other ? mine : other);
                }
            }
        }
    }
}

// One (block, query) candidate buffer: sort its *cnt entries (at most CAP), keep the best kp and
// raise the block's threshold to the kp-th score.  Called by a whole warp; the entries were
// written by threads of the same block before a barrier.
//
// Thresholds are shared between blocks through two arrays.  thr_g_q holds the best known lower
// bound of the query's global kp-th best score (ordered-uint form, atomic max).  top_q[b] holds
// the j-th best score block b has found (j = 1 for kp <= 128, else 2): since blocks scan disjoint
// rows, the r-th largest entry of top_q, r = ceil(kp / j), is exceeded or matched by at least kp
// distinct rows, so it is such a lower bound, and a much tighter one than any single block's
// kp-th best.  With prune set, entries below the shared bound are dropped as well (they cannot
// be among the global best kp).
template <int CAP>
__device__ __noinline__ void warp_compact(u64 *qbuf, int *cnt, float *thr, uint32_t *thr_g_q, int kp,
                                          uint32_t *top_q, int block, int n_blocks, bool prune) {
    const int lane = threadIdx.x & 31;
    const int n = *cnt < CAP ? *cnt : CAP;
    u64 v[CAP / 32];
#pragma unroll
    for (int it = 0; it < CAP / 32; ++it) {
        const int e = it * 32 + lane;
        v[it] = (e < n) ? qbuf[e] : 0ull;
    }
    {
        // cheap first: drop what the shared bound already rules out; if at most kp entries are
        // left, the list need not be sorted (its order does not matter to anyone)
        const uint32_t g0 = __ldcg(thr_g_q);
        int cnt_ge[CAP / 32], ge = 0;
#pragma unroll
        for (int it = 0; it < CAP / 32; ++it) {
            const unsigned mk = __ballot_sync(0xffffffffu, v[it] != 0ull && (uint32_t)(v[it] >> 32) >= g0);
            cnt_ge[it] = ge + __popc(mk & ((1u << lane) - 1u));
            ge += __popc(mk);
        }
        if (ge <= kp && g0 != 0u) {
            __syncwarp();
#pragma unroll
            for (int it = 0; it < CAP / 32; ++it)
                if (v[it] != 0ull && (uint32_t)(v[it] >> 32) >= g0) qbuf[cnt_ge[it]] = v[it];
            __syncwarp();
            if (lane == 0) {
                *cnt = ge;
                const float s = o2f(g0);
                if (s > *thr) *thr = s;
            }
            return;
        }
    }
    warp_sort_desc<CAP / 32>(v);
    int keep = n < kp ? n : kp;
    u64 kth = 0ull;
#pragma unroll
    for (int it = 0; it < CAP / 32; ++it) {
        const int e = it * 32 + lane;
        kth |= (e == kp - 1) ? v[it] : 0ull;             // only the owning lane picks it up
    }
    kth = __shfl_sync(0xffffffffu, kth, (kp - 1) & 31);
    uint32_t bound = (n >= kp) ? (uint32_t)(kth >> 32) : 0u;

    // publish this block's j-th best and derive the bound from all blocks' values
    const int j = (kp + 127) >> 7;
    const int r = (kp + j - 1) / j;
    if (top_q != nullptr && r <= n_blocks && n_blocks <= 256) {
        const uint32_t mine = (uint32_t)(__shfl_sync(0xffffffffu, v[0], j - 1) >> 32);
        if (lane == 0 && n >= j) top_q[block] = mine;
        u64 t[8];
#pragma unroll
        for (int it = 0; it < 8; ++it) {
            const int e = it * 32 + lane;
            uint32_t o = (e < n_blocks) ? __ldcg(&top_q[e]) : 0u;
            if (e == block && n >= j) o = mine;
            t[it] = (u64)o;
        }
        warp_sort_desc<8>(t);
        u64 rth = 0ull;
#pragma unroll
        for (int it = 0; it < 8; ++it) rth |= (it * 32 + lane == r - 1) ? t[it] : 0ull;
        rth = __shfl_sync(0xffffffffu, rth, (r - 1) & 31);
        if ((uint32_t)rth > bound) bound = (uint32_t)rth;
    }
    uint32_t g = bound;
    if (lane == 0 && bound != 0u) {
        const uint32_t old = atomicMax(thr_g_q, bound);
        g = old > bound ? old : bound;
    }
    g = __shfl_sync(0xffffffffu, g, 0);
    if (prune && g != 0u) {
        int ge = 0;
#pragma unroll
        for (int it = 0; it < CAP / 32; ++it)
            ge += __popc(__ballot_sync(0xffffffffu, (uint32_t)(v[it] >> 32) >= g && v[it] != 0ull));
        if (ge < keep) keep = ge;
    }
#pragma unroll
    for (int it = 0; it < CAP / 32; ++it) {
        const int e = it * 32 + lane;
        if (e < keep) qbuf[e] = v[it];
    }
    __syncwarp();
    if (lane == 0) {
        *cnt = keep;
        if (g != 0u) {
            const float s = o2f(g);
            if (s > *thr) *thr = s;
        }
    }
}

// Block-wide bitonic sort of n_pow2 (key, payload) pairs in shared memory, ASCENDING by
// (key, payload).  Call with all threads of the block; n_pow2 is a power of two.
template <typename K, typename V>
__device__ __forceinline__ void block_sort_asc(K *keys, V *vals, int n_pow2) {
    for (int k = 2; k <= n_pow2; k <<= 1) {
        for (int j = k >> 1; j > 0; j >>= 1) {
            __syncthreads();
            for (int e = threadIdx.x; e < n_pow2; e += blockDim.x) {
                const int p = e ^ j;
                if (p > e) {
                    const bool asc = ((e & k) == 0);
                    K ka = keys[e], kb = keys[p];
                    V va = vals[e], vb = vals[p];
                    const bool a_gt_b = (ka > kb) || (ka == kb && va > vb);
                    if (a_gt_b == asc) {
                        keys[e] = kb; keys[p] = ka;
                        vals[e] = vb; vals[p] = va;
                    }
                }
            }
        }
    }
    __syncthreads();
}

}  // namespace prox
