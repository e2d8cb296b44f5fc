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

__device__ __forceinline__ u64 shfl_xor_u64(u64 v, int m) {
    uint32_t lo = __shfl_xor_sync(0xffffffffu, (uint32_t)v, m);
    uint32_t hi = __shfl_xor_sync(0xffffffffu, (uint32_t)(v >> 32), m);
    return ((u64)hi << 32) | lo;
}

// Sorts ITEMS*32 keys held by one warp, DESCENDING.  Element e lives in
// v[e / 32] of lane e % 32, so after the sort v[0] of lane 0 is the largest key,
// v[0] of lane 1 the next, ... v[1] of lane 0 the 33rd, and so on.
template <int ITEMS>
__device__ __forceinline__ void warp_sort_desc(u64 (&v)[ITEMS]) {
    constexpr int LOG = (ITEMS == 1 ? 5 : ITEMS == 2 ? 6 : ITEMS == 4 ? 7 : ITEMS == 8 ? 8 : ITEMS == 16 ? 9 : 10);
    static_assert((32 << (LOG - 5)) == ITEMS * 32, "ITEMS must be a power of two up to 32");
    const int lane = threadIdx.x & 31;
#pragma unroll
    for (int lk = 1; lk <= LOG; ++lk) {
        const int k = 1 << lk;
#pragma unroll
        for (int lj = lk - 1; lj >= 0; --lj) {
            const int j = 1 << lj;
            if (j >= 32) {
                const int dj = j >> 5;
#pragma unroll
                for (int it = 0; it < ITEMS; ++it) {
                    const int partner = it ^ dj;
                    if (partner > it) {
                        const int e = it * 32 + lane;
                        const bool desc = ((e & k) == 0);
                        const u64 a = v[it], b = v[partner];
                        const bool swap = desc ? (a < b) : (a > b);
                        v[it] = swap ? b : a;
                        v[partner] = swap ? a : b;
                    }
                }
            } else {
#pragma unroll
                for (int it = 0; it < ITEMS; ++it) {
                    const int e = it * 32 + lane;
                    const bool desc = ((e & k) == 0);
                    const bool lower = ((lane & j) == 0);       // this lane holds the lower index of the pair
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

// One (block, query) candidate buffer: sort its *cnt entries (at most CAP), keep the best kp,
// raise the block's threshold to the kp-th score and publish it (atomic max on the ordered
// form) for the other blocks.  Called by a whole warp; the entries were written by threads
// of the same block before a barrier.
template <int CAP>
__device__ __forceinline__ void warp_compact(u64 *qbuf, int *cnt, float *thr, uint32_t *thr_g_q, int kp) {
    const int lane = threadIdx.x & 31;
    const int n = *cnt < CAP ? *cnt : CAP;
    u64 v[CAP / 32];
#pragma unroll
    for (int it = 0; it < CAP / 32; ++it) {
        const int e = it * 32 + lane;
        v[it] = (e < n) ? qbuf[e] : 0ull;
    }
    warp_sort_desc<CAP / 32>(v);
    const int keep = n < kp ? n : kp;
    u64 kth = 0ull;
#pragma unroll
    for (int it = 0; it < CAP / 32; ++it) {
        const int e = it * 32 + lane;
        if (e < keep) qbuf[e] = v[it];
        kth |= (e == kp - 1) ? v[it] : 0ull;             // only the owning lane picks it up
    }
    kth = __shfl_sync(0xffffffffu, kth, (kp - 1) & 31);
    __syncwarp();
    if (lane == 0) {
        *cnt = keep;
        if (n >= kp) {
            const float s = entry_score(kth);
            if (s > *thr) *thr = s;
            atomicMax(thr_g_q, (uint32_t)(kth >> 32));
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
