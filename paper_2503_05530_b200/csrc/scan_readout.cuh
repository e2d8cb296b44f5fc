// Accumulator read-out shared by the tensor-core scan kernels: threshold test of 32 accumulator
// columns of one corpus row and ballot-aggregated appends to warp-private candidate lists.
#pragma once
#include "topk_device.cuh"

namespace prox {

// 32 accumulator columns (queries c0 .. c0+31) of one corpus row, one row per lane.
//
// A column passes when acc - thr > half norm, i.e. score = acc - half norm beats the threshold up
// to one rounding (the certificate's slack covers it).  Three levels, cheapest first:
//   1. one maximum over the 32 differences decides the common case that nothing passes;
//   2. else every lane forms its 32 pass bits and one OR across the warp names the columns in
//      which some lane passes;
//   3. only those columns are visited: the passing lanes take consecutive slots of the warp's
//      private list (a ballot replaces atomics) and the warp's best score is folded in.
template <int CAP>
__device__ __forceinline__ void readout32(const uint32_t (&v)[32], int c0, int lc0, float hn, int32_t row,
                                          const float *__restrict__ thr, int *wcnt, uint32_t *best, u64 *lists,
                                          bool &need) {
    float dlt[32];
    float m = -INFINITY;
#pragma unroll
    for (int j4 = 0; j4 < 8; ++j4) {
        const float4 t4 = *reinterpret_cast<const float4 *>(&thr[c0 + 4 * j4]);
        dlt[4 * j4] = __uint_as_float(v[4 * j4]) - t4.x;
        dlt[4 * j4 + 1] = __uint_as_float(v[4 * j4 + 1]) - t4.y;
        dlt[4 * j4 + 2] = __uint_as_float(v[4 * j4 + 2]) - t4.z;
        dlt[4 * j4 + 3] = __uint_as_float(v[4 * j4 + 3]) - t4.w;
        m = fmaxf(m, fmaxf(fmaxf(dlt[4 * j4], dlt[4 * j4 + 1]), fmaxf(dlt[4 * j4 + 2], dlt[4 * j4 + 3])));
    }
    if (!__any_sync(0xffffffffu, m > hn)) return;
    uint32_t pass = 0;
#pragma unroll
    for (int j = 0; j < 32; ++j) pass |= (dlt[j] > hn) ? (1u << j) : 0u;
    const uint32_t cols = __reduce_or_sync(0xffffffffu, pass);
    const int lane = threadIdx.x & 31;
    const unsigned lt = (1u << lane) - 1u;
#pragma unroll
    for (int j = 0; j < 32; ++j) {
        if (cols & (1u << j)) {                                   // warp-uniform
            const bool p = (pass >> j) & 1u;
            const unsigned mask = __ballot_sync(0xffffffffu, p);
            const int base = wcnt[lc0 + j];
            const u64 ent = pack_entry(__uint_as_float(v[j]) - hn, row);
            const int pos = base + __popc(mask & lt);
            if (p && pos < CAP) lists[(size_t)(c0 + j) * CAP + pos] = ent;
            const uint32_t mx = __reduce_max_sync(0xffffffffu, p ? (uint32_t)(ent >> 32) : 0u);
            const int n_new = base + __popc(mask);
            if (lane == 0) {
                wcnt[lc0 + j] = n_new;
                atomicMax(&best[c0 + j], mx);
            }
            if (n_new > CAP - 33) need = true;                    // this list must be cut before the next tile
        }
    }
    __syncwarp();
}

}  // namespace prox
