// Accumulator read-out of the tensor-core scan kernel: threshold test of the accumulator columns
// of one corpus row per lane and ballot-aggregated appends to warp-private candidate lists.
#pragma once
#include "topk_device.cuh"

namespace prox {

// v[j] for a run-time j without indexing the register array: a tree of 31 selects.
__device__ __forceinline__ uint32_t select32(const uint32_t (&v)[32], int j) {
    uint32_t a[16], b[8], c[4], d[2];
#pragma unroll
    for (int i = 0; i < 16; ++i) a[i] = (j & 1) ? v[2 * i + 1] : v[2 * i];
#pragma unroll
    for (int i = 0; i < 8; ++i) b[i] = (j & 2) ? a[2 * i + 1] : a[2 * i];
#pragma unroll
    for (int i = 0; i < 4; ++i) c[i] = (j & 4) ? b[2 * i + 1] : b[2 * i];
#pragma unroll
    for (int i = 0; i < 2; ++i) d[i] = (j & 8) ? c[2 * i + 1] : c[2 * i];
    return (j & 16) ? d[1] : d[0];
}

// Appends of one group of 32 accumulator columns (queries c0 .. c0+31) of one corpus row per
// lane.  Every lane forms its 32 pass bits and walks its own set bits: it takes the next slot of
// the warp's private list of that query with a shared-memory atomic and folds its score into
// the block's best.  Lanes and columns do not wait for one another, so a row that passes for
// many queries at once (queries on one topic) costs a few atomic latencies, and the code stays
// small: this path runs for about one tile in ten and must not crowd the common path out of
// the instruction cache.
template <int CAP>
__device__ __forceinline__ void append32(const uint32_t (&v)[32], int c0, int lc0, float hn, int32_t row,
                                         const float *thr, int *wcnt, uint32_t *best, u64 *lists, bool &need,
                                         int best_stride = 1) {
    uint32_t pass = 0;
#pragma unroll
    for (int j4 = 0; j4 < 8; ++j4) {
        const float4 t4 = *reinterpret_cast<const float4 *>(&thr[c0 + 4 * j4]);
        pass |= (__uint_as_float(v[4 * j4]) - t4.x > hn) ? (1u << (4 * j4)) : 0u;
        pass |= (__uint_as_float(v[4 * j4 + 1]) - t4.y > hn) ? (2u << (4 * j4)) : 0u;
        pass |= (__uint_as_float(v[4 * j4 + 2]) - t4.z > hn) ? (4u << (4 * j4)) : 0u;
        pass |= (__uint_as_float(v[4 * j4 + 3]) - t4.w > hn) ? (8u << (4 * j4)) : 0u;
    }
    bool full = false;
    // While the thresholds are still open (the first tiles of a launch) every row of the quarter
    // passes the same columns.  Then the 32 rows of a column go to 32 consecutive places of its
    // list with one store, the count moves once and the best score is one warp reduction: no
    // per-entry atomics, no register selection, and nothing that orders one column after another.
    const uint32_t pass0 = __shfl_sync(0xffffffffu, pass, 0);
    if (__all_sync(0xffffffffu, pass == pass0) && __popc(pass0) >= 8) {
        const int lane = threadIdx.x & 31;
        const bool mine = (pass0 >> lane) & 1u;                   // lane l keeps the books of column l of the group
        const int base_mine = wcnt[lc0 + lane];
        uint32_t top_mine = 0u;
#pragma unroll
        for (int j = 0; j < 32; ++j) {
            if ((pass0 >> j) & 1u) {                             // warp-uniform
                const u64 ent = pack_entry(__uint_as_float(v[j]) - hn, row);
                const uint32_t top = __reduce_max_sync(0xffffffffu, (uint32_t)(ent >> 32));
                if (lane == j) top_mine = top;
                const int base = __shfl_sync(0xffffffffu, base_mine, j);
                if (base + lane < CAP) lists[(size_t)(c0 + j) * CAP + base + lane] = ent;
            }
        }
        if (mine) {                                              // the warp's columns are its own: plain updates
            wcnt[lc0 + lane] = base_mine + 32;
            uint32_t *bp = best + (size_t)(c0 + lane) * best_stride;      // (stride 1: the block's table; else the shared one)
            if (top_mine > *bp) *bp = top_mine;
        }
        __syncwarp();
        if (__any_sync(0xffffffffu, mine && base_mine + 32 > CAP - 33)) need = true;
        return;
    }
#pragma unroll 1
    while (pass) {
        const int j = __ffs(pass) - 1;
        pass &= pass - 1;
        const u64 ent = pack_entry(__uint_as_float(select32(v, j)) - hn, row);
        const int pos = atomicAdd(&wcnt[lc0 + j], 1);
        if (pos < CAP) lists[(size_t)(c0 + j) * CAP + pos] = ent;
        atomicMax(&best[(size_t)(c0 + j) * best_stride], (uint32_t)(ent >> 32));
        full |= pos + 1 > CAP - 33;                              // this list must be cut before the next tile
    }
    if (__any_sync(0xffffffffu, full)) need = true;
}

// Two fp32 differences with one instruction (sub.f32x2 on register pairs), and the maximum of
// three values with one (max.f32 with three inputs): both are sm_100 forms.  The threshold test
// is the only arithmetic that touches every accumulator, so halving its instruction count
// halves the issue slots the read-out takes.
__device__ __forceinline__ void sub2(uint32_t a0, uint32_t a1, float b0, float b1, float &d0, float &d1) {
    unsigned long long pa, pb, pd;
    asm("mov.b64 %0, {%1, %2};" : "=l"(pa) : "r"(a0), "r"(a1));
    asm("mov.b64 %0, {%1, %2};" : "=l"(pb) : "f"(b0), "f"(b1));
    asm("sub.f32x2 %0, %1, %2;" : "=l"(pd) : "l"(pa), "l"(pb));
    asm("mov.b64 {%0, %1}, %2;" : "=f"(d0), "=f"(d1) : "l"(pd));
}
__device__ __forceinline__ float max3(float a, float b, float c) {
    float m;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(m) : "f"(a), "f"(b), "f"(c));
    return m;
}

// Largest of acc - thr over 32 accumulator columns of this lane's row.
__device__ __forceinline__ float max_margin32(const uint32_t (&v)[32], const float *__restrict__ thr, int c0) {
    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
    for (int j4 = 0; j4 < 8; ++j4) {
        const float4 t4 = *reinterpret_cast<const float4 *>(&thr[c0 + 4 * j4]);
        float d0, d1, d2, d3;
        sub2(v[4 * j4], v[4 * j4 + 1], t4.x, t4.y, d0, d1);
        sub2(v[4 * j4 + 2], v[4 * j4 + 3], t4.z, t4.w, d2, d3);
        m0 = max3(m0, d0, d1);
        m1 = max3(m1, d2, d3);
    }
    return fmaxf(m0, m1);
}

// Largest of 32 accumulator columns of this lane's row, thresholds aside.
__device__ __forceinline__ float raw_max32(const uint32_t (&v)[32]) {
    // four short chains instead of two long ones: the latency of the chain, not the issue slots, is what a tile waits for
    float m0 = max3(__uint_as_float(v[0]), __uint_as_float(v[1]), __uint_as_float(v[2]));
    float m1 = max3(__uint_as_float(v[3]), __uint_as_float(v[4]), __uint_as_float(v[5]));
    float m2 = max3(__uint_as_float(v[6]), __uint_as_float(v[7]), __uint_as_float(v[8]));
    float m3 = max3(__uint_as_float(v[9]), __uint_as_float(v[10]), __uint_as_float(v[11]));
    m0 = max3(m0, __uint_as_float(v[12]), __uint_as_float(v[13]));
    m1 = max3(m1, __uint_as_float(v[14]), __uint_as_float(v[15]));
    m2 = max3(m2, __uint_as_float(v[16]), __uint_as_float(v[17]));
    m3 = max3(m3, __uint_as_float(v[18]), __uint_as_float(v[19]));
    m0 = max3(m0, __uint_as_float(v[20]), __uint_as_float(v[21]));
    m1 = max3(m1, __uint_as_float(v[22]), __uint_as_float(v[23]));
    m2 = max3(m2, __uint_as_float(v[24]), __uint_as_float(v[25]));
    m3 = max3(m3, __uint_as_float(v[26]), __uint_as_float(v[27]));
    m0 = max3(m0, __uint_as_float(v[28]), __uint_as_float(v[29]));
    m1 = max3(m1, __uint_as_float(v[30]), __uint_as_float(v[31]));
    return fmaxf(max3(m0, m1, m2), m3);
}

// Up to 64 accumulator columns (queries c0 .. c0+63; the second 32 only when `two`) of one corpus
// row per lane, already in registers.  A column passes when acc - thr > half norm, i.e. score =
// acc - half norm beats the threshold up to one rounding (the certificate's slack covers it).
// Three levels, cheapest first:
//   1. the row's largest accumulator of a group against the group's smallest threshold (tmin0 /
//      tmin1: lower bounds of the thresholds of the 32 columns, held in registers): no row can
//      pass a column if it does not pass this, and it needs no threshold from shared memory,
//      whose load pipe all read-out warps share;
//   2. for a group that some lane cannot rule out: the per-column margins, one vote;
//   3. the appends.
template <int CAP>
__device__ __forceinline__ void readout64(const uint32_t (&v0)[32], const uint32_t (&v1)[32], bool two, int c0,
                                          int lc0, float hn, float tmin0, float tmin1, int32_t row,
                                          const float *thr, int *wcnt, uint32_t *best, u64 *lists, bool &need,
                                          int best_stride = 1) {
    // (both groups unconditionally, so that their chains overlap; without a second group v1 holds
    // nothing that matters and tmin1 rules it out)
    const float r0 = raw_max32(v0), r1 = raw_max32(v1);
    const bool c0p = r0 - tmin0 > hn;
    const bool c1p = two & (r1 - tmin1 > hn);
    if (!__any_sync(0xffffffffu, c0p | c1p)) return;
    const unsigned maybe0 = __ballot_sync(0xffffffffu, c0p);
    const unsigned maybe1 = __ballot_sync(0xffffffffu, c1p);
    if (maybe0 != 0u) {
        const float m0 = max_margin32(v0, thr, c0);
        if (__any_sync(0xffffffffu, m0 > hn)) append32<CAP>(v0, c0, lc0, hn, row, thr, wcnt, best, lists, need, best_stride);
    }
    if (maybe1 != 0u) {
        const float m1 = max_margin32(v1, thr, c0 + 32);
        if (__any_sync(0xffffffffu, m1 > hn))
            append32<CAP>(v1, c0 + 32, lc0 + 32, hn, row, thr, wcnt, best, lists, need, best_stride);
    }
}

}  // namespace prox
