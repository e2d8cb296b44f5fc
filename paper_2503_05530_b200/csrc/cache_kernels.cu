// Cache-side kernels: the probe (the key distances and their minimum in Algorithm 1, for a whole batch), the
// sequential-order resolve (threshold test, eviction, insertion), and the copies that read and write the value slots.
//
// How a batch is made to behave like B sequential lookups.  During one batch the only
// pre-batch entries that can be evicted are the R = min(B, |C|) entries that come first in
// eviction order (every query causes at most one touch or one eviction, so fewer than B
// entries can leave or be refreshed before the last query).  The probe therefore reduces
// the distances to all other ("safe") slots to one minimum per query, and keeps full rows
// only for the R at-risk slots and for the earlier queries of the same batch.  The resolve
// then replays the batch in index order on those rows alone.
#include <cfloat>
#include <cmath>

#include "prox_internal.h"
#include "topk_device.cuh"

namespace prox {


// ------------------------------------------------------------------------------------------
// At-risk list: the R entries with the smallest stamps, in stamp order (Section 3.3.2: the
// victim is always the entry with the oldest insertion (FIFO) or oldest use (LRU)).
// ------------------------------------------------------------------------------------------
// The R smallest of n unique keys (vals[i], or i when vals is null, rides along), left in
// s_key / s_val (1024 entries each, unused ones at the maximum) for a block of 1024 threads;
// clock bounds the keys from above.  Returns how many were found (R unless the keys repeat).
__device__ int select_smallest(const u64 *__restrict__ keys, const int32_t *__restrict__ vals, long long n, int R,
                               long long clock, unsigned *hist, u64 *s_key, int *s_val, u64 *s_prefix, u64 *s_mask,
                               int *s_remaining, int *s_n) {
    const int tid = threadIdx.x;
    u64 T = ~0ull;                       // R-th smallest key
    if ((long long)R < n) {
        int nd = 1;
        while (nd < 8 && (clock >> (8 * nd)) != 0) ++nd;
        if (tid == 0) { *s_prefix = 0; *s_mask = 0; *s_remaining = R; }
        for (int p = nd - 1; p >= 0; --p) {
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            const u64 prefix = *s_prefix, mask = *s_mask;
            for (long long s = tid; s < n; s += blockDim.x) {
                const u64 v = keys[s];
                if ((v & mask) == prefix) atomicAdd(&hist[(unsigned)(v >> (8 * p)) & 255u], 1u);
            }
            __syncthreads();
            if (tid < 32) {
                int rem = *s_remaining;
                const int b = radix_digit_walk(hist, rem, false);
                if (tid == 0) {
                    *s_remaining = rem;
                    *s_prefix = prefix | ((u64)b << (8 * p));
                    *s_mask = mask | (0xffull << (8 * p));
                }
            }
            __syncthreads();
        }
        T = *s_prefix;
    }
    if (tid == 0) *s_n = 0;
    s_key[tid] = ~0ull;
    s_val[tid] = 0x7fffffff;
    __syncthreads();
    for (long long s = tid; s < n; s += blockDim.x) {
        const u64 v = keys[s];
        if (v <= T) {
            const int pos = atomicAdd(s_n, 1);
            if (pos < 1024) { s_key[pos] = v; s_val[pos] = vals ? vals[s] : (int)s; }
        }
    }
    __syncthreads();
    return *s_n;
}

// Sorts the R selected (stamp, slot) pairs and publishes the at-risk list.
__device__ void publish_risk_list(DevState *st, int R, u64 *s_key, int *s_val, int32_t *risk_pos,
                                  int32_t *risk_slot, u64 *risk_stamp) {
    const int tid = threadIdx.x;
    int n2 = 1;
    while (n2 < R) n2 <<= 1;
    block_sort_asc(s_key, s_val, n2);
    if (tid < R) {
        risk_slot[tid] = s_val[tid];
        risk_stamp[tid] = s_key[tid];
        risk_pos[s_val[tid]] = tid;
    }
    if (tid == 0) {
        st->n_risk = R;
        if (R > 0) st->stamp_floor = (long long)s_key[0];  // stamps only grow: still a lower bound in later batches
    }
}

__device__ __forceinline__ int risk_count(long long count, int B, long long C) {
    return (count + B > C) ? (int)(count < (long long)B ? count : (long long)B) : 0;
}

__global__ void __launch_bounds__(1024)
risk_select_kernel(DevState *st, const u64 *__restrict__ stamp, int32_t *risk_pos,
                   int32_t *risk_slot, u64 *risk_stamp, int B, long long C) {
    __shared__ unsigned hist[256];
    __shared__ u64 s_key[1024];
    __shared__ int s_val[1024];
    __shared__ u64 s_prefix, s_mask;
    __shared__ int s_remaining, s_n;
    const int tid = threadIdx.x;

    const int prev = st->n_risk;
    for (int r = tid; r < prev; r += blockDim.x) risk_pos[risk_slot[r]] = -1;
    const long long count = st->count;
    const long long clock = st->clock;
    __syncthreads();

    const int R = risk_count(count, B, C);
    if (R == 0) {
        if (tid == 0) st->n_risk = 0;
        return;
    }
    const int found = select_smallest(stamp, nullptr, count, R, clock, hist, s_key, s_val, &s_prefix, &s_mask,
                                      &s_remaining, &s_n);
    if (found != R) {                    // stamps must be unique; anything else is a broken state
        if (tid == 0) { atomicCAS(&st->error, 0, PROX_ERR_INTERNAL); st->n_risk = 0; }
        return;
    }
    publish_risk_list(st, R, s_key, s_val, risk_pos, risk_slot, risk_stamp);
}

// Large caches: the same selection spread over the whole GPU.  A 65536-bin histogram of the
// leading bits of (stamp - floor), floor a lower bound of all stored stamps (so that the bins
// cover the range the stamps really span, however long the handle has lived), names the bin
// that holds the R-th smallest; stamps in lower bins are at
// risk for certain, the stamps of that one bin (few, stamps being unique) are settled by one
// block.  Work area: histogram, the two lists and their counters.
constexpr int kRiskBins = 1 << 16;
constexpr int kRiskEdgeCap = 1 << 20;
struct RiskWork {
    unsigned hist[kRiskBins];
    int n_sure, n_edge, bin, shift;
    u64 sure_key[kMaxBatch];
    int32_t sure_val[kMaxBatch];
    u64 edge_key[kRiskEdgeCap];
    int32_t edge_val[kRiskEdgeCap];
};

__device__ __forceinline__ int risk_shift(long long clock) {
    int bits = 0;
    while (bits < 63 && (clock >> bits) != 0) ++bits;
    return bits > 16 ? bits - 16 : 0;
}

__global__ void __launch_bounds__(256)
risk_hist_kernel(const DevState *st, const u64 *__restrict__ stamp, int32_t *risk_pos,
                 const int32_t *__restrict__ risk_slot, RiskWork *w, int B, long long C) {
    const long long gtid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nth = (long long)gridDim.x * blockDim.x;
    const int prev = st->n_risk;
    for (long long r = gtid; r < prev; r += nth) risk_pos[risk_slot[r]] = -1;
    const long long count = st->count;
    const int R = risk_count(count, B, C);
    if (R == 0 || (long long)R >= count) return;
    const u64 floor = (u64)st->stamp_floor;
    const int shift = risk_shift(st->clock - (long long)floor);
    for (long long s = gtid; s < count; s += nth) atomicAdd(&w->hist[(unsigned)((stamp[s] - floor) >> shift)], 1u);
}

__global__ void __launch_bounds__(1024)
risk_pick_kernel(const DevState *st, RiskWork *w, int B, long long C) {
    __shared__ unsigned part[1024];
    const int tid = threadIdx.x;
    const long long count = st->count;
    const int R = risk_count(count, B, C);
    if (tid == 0) { w->n_sure = 0; w->n_edge = 0; w->shift = risk_shift(st->clock - st->stamp_floor); }
    if (R == 0 || (long long)R >= count) {
        if (tid == 0) w->bin = kRiskBins;                // every entry (or none) is at risk
        return;
    }
    // sums of 64 consecutive bins, one group per warp at a time (coalesced), then the group and the
    // bin inside it where the running count reaches R
    constexpr int per = kRiskBins / 1024;
    static_assert(per == 64, "two coalesced loads per lane cover one group");
    __shared__ unsigned s_acc;
    __shared__ int s_group;
    const int lane = tid & 31, warp = tid >> 5;
    for (int g = warp; g < 1024; g += 32) {
        unsigned v = w->hist[g * per + lane] + w->hist[g * per + 32 + lane];
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) v += __shfl_xor_sync(0xffffffffu, v, m);
        if (lane == 0) part[g] = v;
    }
    __syncthreads();
    // the first group whose running count reaches R (the last group if none does): running counts by a
    // block-wide prefix sum; they only grow, so the group is the number of groups that stay below R
    __shared__ unsigned wt[32];
    unsigned incl = part[tid];
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const unsigned y = __shfl_up_sync(0xffffffffu, incl, m);
        if (lane >= m) incl += y;
    }
    if (lane == 31) wt[warp] = incl;
    if (tid == 0) s_acc = 0;
    __syncthreads();
    if (warp == 0) {
        unsigned v = wt[lane];
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
            const unsigned y = __shfl_up_sync(0xffffffffu, v, m);
            if (lane >= m) v += y;
        }
        wt[lane] = v;
    }
    __syncthreads();
    if (warp > 0) incl += wt[warp - 1];
    int t = __syncthreads_count(incl < (unsigned)R);
    if (t > 1023) t = 1023;
    if (tid == t - 1) s_acc = incl;                      // the count before group t
    if (tid == 0) s_group = t;
    __syncthreads();
    // the same inside the group's 64 bins, by one warp (two bins a lane)
    if (warp == 0) {
        const unsigned f0 = w->hist[t * per + 2 * lane], f1 = w->hist[t * per + 2 * lane + 1];
        unsigned in2 = f0 + f1;
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
            const unsigned y = __shfl_up_sync(0xffffffffu, in2, m);
            if (lane >= m) in2 += y;
        }
        const unsigned before = s_acc + in2 - f0 - f1;
        int i = __popc(__ballot_sync(0xffffffffu, before + f0 < (unsigned)R)) +
                __popc(__ballot_sync(0xffffffffu, before + f0 + f1 < (unsigned)R));
        if (i > per - 1) i = per - 1;
        if (lane == 0) w->bin = t * per + i;
    }
}

__global__ void __launch_bounds__(256)
risk_collect_kernel(const DevState *st, const u64 *__restrict__ stamp, RiskWork *w, int B, long long C) {
    const long long count = st->count;
    if (risk_count(count, B, C) == 0) return;
    const long long gtid = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    const long long nth = (long long)gridDim.x * blockDim.x;
    const unsigned bin = (unsigned)w->bin;
    const int shift = w->shift;
    const u64 floor = (u64)st->stamp_floor;
    for (long long s = gtid; s < count; s += nth) {
        const u64 v = stamp[s];
        const unsigned bn = bin == (unsigned)kRiskBins ? 0u : (unsigned)((v - floor) >> shift);
        if (bn < bin) {
            const int pos = atomicAdd(&w->n_sure, 1);
            if (pos < kMaxBatch) { w->sure_key[pos] = v; w->sure_val[pos] = (int32_t)s; }
        } else if (bn == bin) {
            const int pos = atomicAdd(&w->n_edge, 1);
            if (pos < kRiskEdgeCap) { w->edge_key[pos] = v; w->edge_val[pos] = (int32_t)s; }
        }
    }
}

__global__ void __launch_bounds__(1024)
risk_finish_kernel(DevState *st, RiskWork *w, int32_t *risk_pos, int32_t *risk_slot, u64 *risk_stamp, int B,
                   long long C) {
    __shared__ unsigned hist[256];
    __shared__ u64 s_key[1024];
    __shared__ int s_val[1024];
    __shared__ u64 s_prefix, s_mask;
    __shared__ int s_remaining, s_n;
    const int tid = threadIdx.x;
    const long long count = st->count;
    const int R = risk_count(count, B, C);
    if (R == 0) {
        if (tid == 0) st->n_risk = 0;
        return;
    }
    const int n_sure = w->n_sure, n_edge = w->n_edge;
    const int need = R - n_sure;
    bool ok = n_sure <= R && need <= n_edge && n_edge <= kRiskEdgeCap;
    int found = 0;
    if (ok) {
        found = need > 0 ? select_smallest(w->edge_key, w->edge_val, n_edge, need, st->clock, hist, s_key, s_val,
                                           &s_prefix, &s_mask, &s_remaining, &s_n)
                         : 0;
        if (need <= 0) {
            s_key[tid] = ~0ull;
            s_val[tid] = 0x7fffffff;
            __syncthreads();
        }
        ok = found == (need > 0 ? need : 0);
    }
    if (!ok) {                           // stamps must be unique; anything else is a broken state
        if (tid == 0) { atomicCAS(&st->error, 0, PROX_ERR_INTERNAL); st->n_risk = 0; }
        return;
    }
    if (tid < n_sure) { s_key[found + tid] = w->sure_key[tid]; s_val[found + tid] = w->sure_val[tid]; }
    __syncthreads();
    publish_risk_list(st, R, s_key, s_val, risk_pos, risk_slot, risk_stamp);
}

// FIFO needs no selection: slots fill in index order and a victim's slot is reused by the entry
// that replaces it, so the stored entries form a ring in insertion order, and the R oldest are the
// R slots from the ring's head on (Section 3.3.2: FIFO evicts the oldest inserted entry).
__global__ void __launch_bounds__(1024)
risk_ring_kernel(DevState *st, const u64 *__restrict__ stamp, int32_t *risk_pos, int32_t *risk_slot,
                 u64 *risk_stamp, int B, long long C) {
    const int tid = threadIdx.x;
    const int prev = st->n_risk;
    for (int r = tid; r < prev; r += blockDim.x) risk_pos[risk_slot[r]] = -1;
    const long long count = st->count, head = st->fifo_head;
    __syncthreads();
    const int R = risk_count(count, B, C);
    if (tid < R) {
        const long long slot = (head + tid) % count;
        risk_slot[tid] = (int32_t)slot;
        risk_stamp[tid] = stamp[slot];
        risk_pos[slot] = tid;
    }
    if (tid == 0) st->n_risk = R;
}

// ------------------------------------------------------------------------------------------
// Probe: squared distances, in fp64 over the fp32 values and in difference form (so that a
// bitwise duplicate is at distance exactly 0), from each query to every valid key and to
// every earlier query of the batch.  IP = true: the inner product as a distance, -(q . key),
// an fp64 sum of the products.  Tile: 32 queries x 64 (or 32) columns per block, d in chunks of 32 (or 64).
//   mode 0  columns = slots [0, count) then the batch [count, count + B): everything in fp64.
//   mode 1  columns = the R at-risk slots then the batch: what the resolve needs as full rows
//           when the safe slots are handled by the coarse tensor-core probe.
//   mode 2  queries = those the coarse probe could not certify (pfail_list), columns = slots.
//   mode 3  columns = slots only, the at-risk ones left out: the safe minimum alone (the at-risk
//           slots and the batch go through the tensor-core pass of probe_side.cu).
//   mode 4  mode 1, but only if that pass listed more pairs than it can hold (else return at once).
// ------------------------------------------------------------------------------------------
constexpr int PQ = 32;
constexpr int kProbeColsWide = 64, kProbeColsNarrow = 32, kProbeColsTiny = 16;

// PC = columns per block tile, PD = dimensions per step: 64 x 32, or 32 x 64 for a small cache,
// where the wide tiles leave most SMs without a block and the time goes into the chain of steps
// (a barrier and a load latency each): narrower tiles give twice the blocks, deeper steps half
// the chain with twice the loads in flight.
template <int PC, int PD, bool IP>
__global__ void __launch_bounds__(256)
probe_kernel(const DevState *__restrict__ st, const float *__restrict__ keys,
             const float *__restrict__ queries, const int32_t *__restrict__ risk_pos, int B, int d,
             double *__restrict__ part_min, int32_t *__restrict__ part_arg,
             double *__restrict__ d_risk, double *__restrict__ d_intra, int mode,
             const int32_t *__restrict__ risk_slot, const int32_t *__restrict__ pfail_list) {
    __shared__ double qs[PQ][PD + 1];
    __shared__ double ks[PC][PD + 1];
    __shared__ int q_index[PQ];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
    if (mode == 4) {
        if (!st->side_overflow) return;
        mode = 1;
    }
    const long long count = st->count;
    const int R = st->n_risk;
    const int nq = mode == 2 ? st->n_pfail : B;            // queries this launch serves
    if ((int)blockIdx.x * PQ >= nq) return;
    const long long nslot_cols = mode == 1 ? R : count;      // columns that are cached keys
    const long long ncols = (mode == 2 || mode == 3) ? count : nslot_cols + B;
    if (tid < PQ) {
        const int r = blockIdx.x * PQ + tid;
        q_index[tid] = r < nq ? (mode == 2 ? pfail_list[r] : r) : -1;
    }
    __syncthreads();
    const long long ntiles = (ncols + PC - 1) / PC;
    const int S = gridDim.y, sp = blockIdx.y;
    const long long per = (ntiles + S - 1) / S;
    const long long t_begin = sp * per;
    const long long t_end = (t_begin + per < ntiles) ? t_begin + per : ntiles;
    double best_d[2] = {INFINITY, INFINITY};
    int best_s[2] = {0x7fffffff, 0x7fffffff};

    for (long long t = t_begin; t < t_end; ++t) {
        const long long c0 = t * PC;
        double acc[2][PC / 16];
#pragma unroll
        for (int a = 0; a < 2; ++a)
#pragma unroll
            for (int b = 0; b < PC / 16; ++b) acc[a][b] = 0.0;

        // operands of the next 32 dimensions are fetched into registers while the current ones are
        // multiplied: small problems (few blocks per SM) are bound by this latency, not by the fp64 rate
        const float *q_src[(PQ * PD) / 256];
        const float *k_src[(PC * PD) / 256];
#pragma unroll
        for (int it = 0; it < (PQ * PD) / 256; ++it) {
            const int idx = it * 256 + tid, r = idx / PD, c = idx % PD;
            const int qi = q_index[r];
            q_src[it] = qi >= 0 ? queries + (size_t)qi * d + c : nullptr;
        }
#pragma unroll
        for (int it = 0; it < (PC * PD) / 256; ++it) {
            const int idx = it * 256 + tid, r = idx / PD, c = idx % PD;
            const long long col = c0 + r;
            k_src[it] = nullptr;
            if (col < ncols)
                k_src[it] = ((col >= nslot_cols) ? queries + (size_t)(col - nslot_cols) * d
                                                 : keys + (size_t)(mode == 1 ? risk_slot[col] : col) * d) + c;
        }
        float q_next[(PQ * PD) / 256], k_next[(PC * PD) / 256];
#pragma unroll
        for (int it = 0; it < (PQ * PD) / 256; ++it)
            q_next[it] = (q_src[it] && (it * 256 + tid) % PD < d) ? q_src[it][0] : 0.f;
#pragma unroll
        for (int it = 0; it < (PC * PD) / 256; ++it)
            k_next[it] = (k_src[it] && (it * 256 + tid) % PD < d) ? k_src[it][0] : 0.f;

        for (int kc = 0; kc < d; kc += PD) {
            __syncthreads();
#pragma unroll
            for (int it = 0; it < (PQ * PD) / 256; ++it) {
                const int idx = it * 256 + tid, r = idx / PD, c = idx % PD;
                qs[r][c] = (double)q_next[it];
            }
#pragma unroll
            for (int it = 0; it < (PC * PD) / 256; ++it) {
                const int idx = it * 256 + tid, r = idx / PD, c = idx % PD;
                ks[r][c] = (double)k_next[it];
            }
            __syncthreads();
            {
                const int kn = kc + PD;
#pragma unroll
                for (int it = 0; it < (PQ * PD) / 256; ++it)
                    q_next[it] = (q_src[it] && kn + (it * 256 + tid) % PD < d) ? q_src[it][kn] : 0.f;
#pragma unroll
                for (int it = 0; it < (PC * PD) / 256; ++it)
                    k_next[it] = (k_src[it] && kn + (it * 256 + tid) % PD < d) ? k_src[it][kn] : 0.f;
            }
#pragma unroll 8
            for (int j = 0; j < PD; ++j) {
                const double qa = qs[ty * 2][j], qb2 = qs[ty * 2 + 1][j];
#pragma unroll
                for (int b = 0; b < PC / 16; ++b) {
                    const double kv = ks[tx + 16 * b][j];
                    if constexpr (IP) {
                        acc[0][b] = fma(-qa, kv, acc[0][b]);
                        acc[1][b] = fma(-qb2, kv, acc[1][b]);
                    } else {
                        const double d0 = qa - kv, d1 = qb2 - kv;
                        acc[0][b] = fma(d0, d0, acc[0][b]);
                        acc[1][b] = fma(d1, d1, acc[1][b]);
                    }
                }
            }
        }
#pragma unroll
        for (int a = 0; a < 2; ++a) {
            const int i = q_index[ty * 2 + a];
            if (i < 0) continue;
#pragma unroll
            for (int b = 0; b < PC / 16; ++b) {
                const long long col = c0 + tx + 16 * b;
                if (col >= ncols) continue;
                const double v = acc[a][b];
                if (col < nslot_cols) {
                    const int rp = mode == 1 ? (int)col : risk_pos[col];
                    if (rp >= 0) {
                        if (mode < 2) d_risk[(size_t)i * kMaxBatch + rp] = v;
                    } else if (v < best_d[a] || (v == best_d[a] && (int)col < best_s[a])) {
                        best_d[a] = v;
                        best_s[a] = (int)col;
                    }
                } else {
                    const int j = (int)(col - nslot_cols);
                    if (j < i) d_intra[(size_t)i * kMaxBatch + j] = v;
                }
            }
        }
    }
    // minimum over the 16 threads that share a query (lanes of one half warp)
#pragma unroll
    for (int a = 0; a < 2; ++a) {
#pragma unroll
        for (int m = 1; m < 16; m <<= 1) {
            const double od = __shfl_xor_sync(0xffffffffu, best_d[a], m);
            const int os = __shfl_xor_sync(0xffffffffu, best_s[a], m);
            if (od < best_d[a] || (od == best_d[a] && os < best_s[a])) { best_d[a] = od; best_s[a] = os; }
        }
        const int i = q_index[ty * 2 + a];
        if (tx == 0 && i >= 0 && mode != 1) {
            part_min[(size_t)i * kProbeSplitMax + sp] = best_d[a];
            part_arg[(size_t)i * kProbeSplitMax + sp] = best_s[a];
        }
    }
}

// ------------------------------------------------------------------------------------------
// Per query: reduce the partial safe minima; list the at-risk and in-batch keys within tau
// (the threshold test of Algorithm 1, inclusive), nearest first.  code < kMaxBatch: at-risk
// position; else kMaxBatch + j.  The list is sorted by (distance, code) so that the replay only
// has to find the first entry that is still resident.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
build_candidates_kernel(const DevState *__restrict__ st, int B, int S, double tau,
                        const double *__restrict__ part_min, const int32_t *__restrict__ part_arg,
                        const double *__restrict__ d_risk, const double *__restrict__ d_intra,
                        double *safe_min, int32_t *safe_arg, double *cand_d, int32_t *cand_code,
                        int32_t *n_cand, const int32_t *__restrict__ use_partial, int lists_ready) {
    __shared__ int s_n;
    __shared__ double s_d[2 * kMaxBatch];
    __shared__ int s_code[2 * kMaxBatch];
    const int i = blockIdx.x, tid = threadIdx.x;
    if (i >= B) return;
    if (tid == 0) s_n = 0;
    __syncthreads();
    if (tid < 32 && (use_partial == nullptr || use_partial[i])) {   // else the coarse probe has set them
        double bd = INFINITY;
        int bs = 0x7fffffff;
        for (int s = tid; s < S; s += 32) {
            const double v = part_min[(size_t)i * kProbeSplitMax + s];
            const int a = part_arg[(size_t)i * kProbeSplitMax + s];
            if (v < bd || (v == bd && a < bs)) { bd = v; bs = a; }
        }
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
            const double od = __shfl_xor_sync(0xffffffffu, bd, m);
            const int os = __shfl_xor_sync(0xffffffffu, bs, m);
            if (od < bd || (od == bd && os < bs)) { bd = od; bs = os; }
        }
        if (tid == 0) {
            safe_min[i] = bd;
            safe_arg[i] = (bs == 0x7fffffff) ? -1 : bs;
        }
    }
    const int R = st->n_risk;
    const size_t base = (size_t)i * (2 * kMaxBatch);
    if (lists_ready && !st->side_overflow) {              // the pairs within tau are listed already: only sort them
        const int nl = n_cand[i];
        for (int e = tid; e < nl; e += blockDim.x) { s_d[e] = cand_d[base + e]; s_code[e] = cand_code[base + e]; }
        if (tid == 0) s_n = nl;
    } else {
        for (int e = tid; e < R + i; e += blockDim.x) {
            double v;
            int code;
            if (e < R) { v = d_risk[(size_t)i * kMaxBatch + e]; code = e; }
            else { v = d_intra[(size_t)i * kMaxBatch + (e - R)]; code = kMaxBatch + (e - R); }
            if (v <= tau) {
                const int pos = atomicAdd(&s_n, 1);
                s_d[pos] = v;
                s_code[pos] = code;
            }
        }
    }
    __syncthreads();
    const int n = s_n;
    if (n > 1) {                                          // (block-uniform)
        int n2 = 2;
        while (n2 < n) n2 <<= 1;
        for (int e = n + tid; e < n2; e += blockDim.x) { s_d[e] = INFINITY; s_code[e] = 0x7fffffff; }
        block_sort_asc(s_d, s_code, n2);
    }
    for (int e = tid; e < n; e += blockDim.x) {
        cand_d[base + e] = s_d[e];
        cand_code[base + e] = s_code[e];
    }
    if (tid == 0) n_cand[i] = n;
}

// ------------------------------------------------------------------------------------------
// Resolve: replay queries 0..B-1 in order (Algorithm 1 from the threshold test to the insertion).
// One block.  Three kinds of query:
//   settled     no at-risk or in-batch key within tau, nearest safe key within tau: a hit on that
//               key whatever the rest of the batch does; answered in parallel while loading;
//   plain miss  no key of any kind within tau: a miss for certain; it only has to take its slot
//               in order;
//   entangled   some at-risk or in-batch key within tau: hit or miss depends on which of them are
//               still resident when its turn comes.
// Warp 0 walks the entangled queries in order; the plain misses between two of them are settled
// 32 at a time (free slots first, then the next at-risk entries that nobody touched, found by
// one vote per 32 entries).  An entangled query finds the first resident entry of its sorted list
// with one vote per 32 entries.  Only when the at-risk list is used up (a capacity below the
// batch size) does a miss search all refreshed and in-batch entries for the oldest stamp.
// ------------------------------------------------------------------------------------------
constexpr int kCsrCap = 8192;

struct ResolveSmem {
    u64 r_stamp[kMaxBatch];
    u64 b_stamp[kMaxBatch];
    double safe_min[kMaxBatch];
    double csr_d[kCsrCap];
    int csr_code[kCsrCap];
    int r_slot[kMaxBatch];
    int b_slot[kMaxBatch];
    int safe_arg[kMaxBatch];
    int ncand[kMaxBatch];
    int off[kMaxBatch + 1];
    int plain_list[kMaxBatch];         // the plain misses in index order
    int ent_list[kMaxBatch];           // the entangled queries in index order
    int plain_before[kMaxBatch];       // per entangled query (by its place in ent_list): plain misses before it
    int warp_tot[3][32];
    int one[1];
    int head[kMaxBatch];               // first entry of the query's list that may still be a resident key
    unsigned char kind[kMaxBatch];     // 1 settled (hits a safe key), 2 plain miss, 3 entangled
    unsigned char r_alive[kMaxBatch];
    unsigned char r_touched[kMaxBatch];
    // the parallel replay (replay_parallel)
    int p_tgt[kMaxBatch];              // per query: -1 miss, -2 its nearest safe key, h >= 0 the h-th entry of its list
    int p_tm[kMaxBatch];               // query index of the m-th evicting miss
    int p_E[kMaxBatch];                // per at-risk position: the query that evicts it (kNever: none)
    int p_T[kMaxBatch];                // per at-risk position: the first query that hits it; at the end, the position the m-th eviction takes
    unsigned char p_skip[kMaxBatch];   // per at-risk position: touched before the eviction pointer reaches it
    int p_flag;                        // a case the parallel replay leaves to the sequential one
};

struct ReplayState {
    long long cnt;                     // |C| so far
    int p;                             // first at-risk position that may still be untouched and resident
    int n_miss, n_evict;
};

struct ResolveOut {
    uint8_t *out_hit;
    int32_t *src, *src_kind, *evt_slot, *miss_list, *miss_rank;
    float *evt_dist;
};

// Position of the n-th set bit of mask (n counted from 0; mask has more than n bits set): five
// halvings with a population count each.
__device__ __forceinline__ int nth_set_bit(unsigned mask, int n) {
    int pos = 0;
#pragma unroll
    for (int s = 16; s >= 1; s >>= 1) {
        const int c = __popc(mask & (((1u << s) - 1u) << pos));
        if (n >= c) { n -= c; pos += s; }
    }
    return pos;
}

// The misses list[a .. b) (query indices, ascending) take their slots in order.  Whole warp.
__device__ void settle_misses(ResolveSmem &sm, ReplayState &rs, const int *list, int a, int b, int R, long long C,
                              long long clock0, DevState *st, const ResolveOut &o) {
    const int lane = threadIdx.x & 31;
    for (int base = a; base < b; base += 32) {
        const int m = b - base < 32 ? b - base : 32;
        const int i = lane < m ? list[base + lane] : -1;
        const long long free_now = C - rs.cnt;
        const int n_free = free_now <= 0 ? 0 : (free_now < m ? (int)free_now : m);
        int slot = -1;
        if (lane < n_free) slot = (int)(rs.cnt + lane);
        rs.cnt += n_free;
        const int need = m - n_free;
        int got = 0;
        while (got < need && rs.p < R) {                   // the next 32 at-risk entries
            const int e = rs.p + lane;
            const bool ok = e < R && sm.r_alive[e] && !sm.r_touched[e];
            const unsigned mask = __ballot_sync(0xffffffffu, ok);
            const int avail = __popc(mask);
            const int use = avail < need - got ? avail : need - got;
            const int t = lane - n_free - got;             // this lane's turn among the evicting misses
            if (t >= 0 && t < use) slot = sm.r_slot[rs.p + nth_set_bit(mask, t)];
            if (ok && __popc(mask & ((1u << lane) - 1u)) < use) sm.r_alive[e] = 0;
            got += use;
            rs.p = (use == avail) ? rs.p + 32 : rs.p + nth_set_bit(mask, use - 1) + 1;
            __syncwarp();
        }
        if (rs.p > R) rs.p = R;
        rs.n_evict += got;
        const int n_fast = n_free + got;
        if (lane < n_fast) {
            const int rank = rs.n_miss + lane;
            o.out_hit[i] = 0; o.src_kind[i] = 0; o.src[i] = -1;
            o.evt_slot[i] = slot; o.evt_dist[i] = INFINITY;
            sm.b_slot[i] = slot; sm.b_stamp[i] = (u64)(clock0 + i);
            o.miss_list[rank] = i; o.miss_rank[i] = rank;
        }
        __syncwarp();
        // the at-risk list is used up: each remaining miss evicts the oldest of the refreshed at-risk
        // entries and of the entries this batch inserted before it
        for (int t = n_fast; t < m; ++t) {
            const int ii = __shfl_sync(0xffffffffu, i, t);
            u64 bs = ~0ull;
            int bc = -1;
            for (int e = lane; e < R + ii; e += 32) {
                u64 v;
                bool ok;
                if (e < R) { ok = sm.r_alive[e] != 0; v = sm.r_stamp[e]; }
                else { ok = sm.b_slot[e - R] >= 0; v = sm.b_stamp[e - R]; }
                if (ok && v < bs) { bs = v; bc = e; }
            }
#pragma unroll
            for (int mm = 1; mm < 32; mm <<= 1) {
                const u64 ov = __shfl_xor_sync(0xffffffffu, bs, mm);
                const int oc = __shfl_xor_sync(0xffffffffu, bc, mm);
                if (ov < bs) { bs = ov; bc = oc; }
            }
            int vslot = 0;
            if (bc < 0) {                                  // cannot happen with capacity >= 1
                if (lane == 0) atomicCAS(&st->error, 0, PROX_ERR_INTERNAL);
            } else if (bc < R) {
                vslot = sm.r_slot[bc];
                if (lane == 0) sm.r_alive[bc] = 0;
            } else {
                vslot = sm.b_slot[bc - R];
                if (lane == 0) sm.b_slot[bc - R] = -1;
            }
            __syncwarp();
            if (lane == 0) {
                const int rank = rs.n_miss + t;
                o.out_hit[ii] = 0; o.src_kind[ii] = 0; o.src[ii] = -1;
                o.evt_slot[ii] = vslot; o.evt_dist[ii] = INFINITY;
                sm.b_slot[ii] = vslot; sm.b_stamp[ii] = (u64)(clock0 + ii);
                o.miss_list[rank] = ii; o.miss_rank[ii] = rank;
            }
            rs.n_evict++;
            __syncwarp();
        }
        rs.n_miss += m;
    }
}

// Exclusive prefix sum of x over the block's 1024 threads (wt: 32 ints of shared memory); total = the sum.
__device__ __forceinline__ int block_excl_scan(int x, int *wt, int &total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = x;
#pragma unroll
    for (int m = 1; m < 32; m <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, inc, m);
        if (lane >= m) inc += y;
    }
    if (lane == 31) wt[warp] = inc;
    __syncthreads();
    if (warp == 0) {
        int w = wt[lane];
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, w, m);
            if (lane >= m) w += y;
        }
        wt[lane] = w;
    }
    __syncthreads();
    total = wt[31];
    const int r = inc - x + (warp > 0 ? wt[warp - 1] : 0);
    __syncthreads();                                       // wt is free again
    return r;
}

// The replay of Algorithm 1 over one batch as a fixed point, for batches in which many queries
// depend on one another (a cache about as small as the batch: every key is at risk).
//
// The outcome of query i (miss, or the key it hits) depends only on what the queries before it
// did: which at-risk keys they evicted and which of them were inserted.  Write that as equations
// over the whole batch:
//   rank(i)  = misses before i; the misses of rank >= free slots evict, in order;
//   T(q)     = the first query that hits at-risk position q (LRU only: a touched key moves to
//              the young end and the eviction pointer passes over it);
//   m(q)     = positions before q that the pointer does not pass over; position q is passed
//              over iff T(q) is earlier than the (m(q)+1)-th evicting miss, and evicted by that
//              miss otherwise: E(q);
//   query i hits the first entry of its sorted list that is resident when it arrives: an at-risk
//              position q with E(q) >= i (the miss that evicts q found it resident), or a query
//              j < i that missed (and so was inserted); else its safe key within tau; else it misses.
// Every right-hand side at "time" i uses only outcomes of earlier times, so the system has one
// solution, the sequential replay, and iterating all equations in parallel from any start makes
// at least the earliest wrong outcome right in each round.  In practice a batch of 1024 settles
// in 5 to 13 rounds.  The iteration stops when a round changes nothing.
//
// Left to the sequential replay (returns false, nothing written): two listed keys, or a listed
// and the safe key, at exactly the same distance (the lowest slot wins, and slots of inserted keys
// are not part of the equations); more evictions than at-risk positions (capacity below the
// batch size); no fixed point within kParallelRounds.
constexpr int kNever = 0x7fffffff;
constexpr int kParallelRounds = 48;
constexpr int kParallelMinEntangled = 24;

__device__ bool replay_parallel(ResolveSmem &sm, DevState *st, int B, int R, long long C, double tau, int policy,
                                long long count0, long long clock0, const double *cand_d, const int32_t *cand_code,
                                u64 *stamp, const ResolveOut &o) {
    const int i = threadIdx.x;
    const bool lru = policy == PROX_LRU;
    const long long free_ll = C - count0;
    const int free0 = free_ll <= 0 ? 0 : (free_ll > (long long)B ? B : (int)free_ll);
    const int kind = i < B ? (int)sm.kind[i] : 0;
    int n = 0, hd = 0, sa = -1;
    double sd = INFINITY;
    const int *lc = nullptr;
    const double *ld = nullptr;
    if (i < B) {
        n = sm.ncand[i];
        hd = sm.head[i];
        sd = sm.safe_min[i];
        sa = sm.safe_arg[i];
        const int off = sm.off[i];
        const bool in_smem = off + n <= kCsrCap;
        lc = in_smem ? sm.csr_code + off : cand_code + (size_t)i * (2 * kMaxBatch);
        ld = in_smem ? sm.csr_d + off : cand_d + (size_t)i * (2 * kMaxBatch);
    }
    const bool safe_hit = sa >= 0 && sd <= tau;
    // start: every listed key is taken as resident
    if (i < B) sm.p_tgt[i] = kind == 2 ? -1 : (kind == 1 ? -2 : hd);
    if (i < kMaxBatch) { sm.p_skip[i] = 0; sm.p_E[i] = kNever; }
    if (i == 0) sm.p_flag = 0;
    __syncthreads();

    int rank = 0, total_miss = 0, mq = 0, total_ev = 0;
    bool is_miss = false, converged = false;
    for (int round = 0; round < kParallelRounds; ++round) {
        is_miss = i < B && sm.p_tgt[i] == -1;
        rank = block_excl_scan(is_miss ? 1 : 0, sm.warp_tot[0], total_miss);
        if (i < kMaxBatch) { sm.p_tm[i] = kNever; sm.p_T[i] = kNever; }
        __syncthreads();
        if (is_miss && rank >= free0) sm.p_tm[rank - free0] = i;
        if (lru && kind == 3) {
            const int t = sm.p_tgt[i];
            if (t >= 0) {
                const int code = lc[t];
                if (code < kMaxBatch) atomicMin(&sm.p_T[code], i);
            }
        }
        mq = block_excl_scan((i < R && !sm.p_skip[i]) ? 1 : 0, sm.warp_tot[1], total_ev);   // (its barriers order the writes above)
        bool changed = false;
        if (i < R) {
            const int et = sm.p_tm[mq];                     // mq < R <= kMaxBatch
            const bool skip = sm.p_T[i] < et;
            const int E = skip ? kNever : et;
            if ((skip ? 1 : 0) != (int)sm.p_skip[i] || E != sm.p_E[i]) changed = true;
            sm.p_skip[i] = skip ? 1 : 0;
            sm.p_E[i] = E;
        }
        __syncthreads();
        if (kind == 3) {
            int t = -1;
            for (int h = hd; h < n; ++h) {
                const int code = lc[h];
                // (outcomes of other queries are read while their threads may be writing this sweep's:
                // either value is a legitimate iterate, and a sweep that changes nothing read only final ones)
                const bool valid = code < kMaxBatch ? sm.p_E[code] >= i
                                                    : ((volatile int *)sm.p_tgt)[code - kMaxBatch] == -1;
                if (valid) { t = h; break; }
            }
            if (t >= 0) {
                const double bd = ld[t];
                if (t + 1 < n && ld[t + 1] == bd) sm.p_flag = 1;
                if (safe_hit) {
                    if (sd < bd) t = -2;
                    else if (sd == bd) sm.p_flag = 1;
                }
            } else if (safe_hit) {
                t = -2;
            }
            if (t != sm.p_tgt[i]) { sm.p_tgt[i] = t; changed = true; }
        }
        const int any = __syncthreads_or(changed ? 1 : 0);
        if (sm.p_flag) return false;
        if (!any) { converged = true; break; }
    }
    if (!converged) return false;
    // (rank, total_miss, mq, total_ev, p_tm, p_skip, p_E are those of the last sweep, which changed nothing)
    const int n_evict = total_miss > free0 ? total_miss - free0 : 0;
    if (n_evict > total_ev) return false;                  // the at-risk list would be used up
    const int n_free = total_miss < free0 ? total_miss : free0;

    if (i < R && !sm.p_skip[i] && mq < n_evict) { sm.p_T[mq] = i; sm.r_alive[i] = 0; }
    __syncthreads();
    if (is_miss) {
        const int slot = rank < free0 ? (int)(count0 + rank) : sm.r_slot[sm.p_T[rank - free0]];
        o.out_hit[i] = 0; o.src_kind[i] = 0; o.src[i] = -1;
        o.evt_slot[i] = slot; o.evt_dist[i] = INFINITY;
        sm.b_slot[i] = slot; sm.b_stamp[i] = (u64)(clock0 + i);
        o.miss_list[rank] = i; o.miss_rank[i] = rank;
    }
    __syncthreads();
    int intra = 0;
    if (kind == 3 && !is_miss) {
        const u64 t = (u64)(clock0 + i);
        const int h = sm.p_tgt[i];
        o.out_hit[i] = 1;
        o.miss_rank[i] = -1;
        if (h == -2) {
            o.evt_slot[i] = sa; o.evt_dist[i] = (float)sd;
            o.src_kind[i] = 1; o.src[i] = sa;
            if (lru) atomicMax(&stamp[sa], t);
        } else {
            const int code = lc[h];
            o.evt_dist[i] = (float)ld[h];
            if (code < kMaxBatch) {
                const int slot = sm.r_slot[code];
                o.evt_slot[i] = slot;
                o.src_kind[i] = 1; o.src[i] = slot;
                if (lru) { atomicMax(&sm.r_stamp[code], t); sm.r_touched[code] = 1; }
            } else {
                const int j = code - kMaxBatch;
                o.evt_slot[i] = sm.b_slot[j];
                o.src_kind[i] = 2; o.src[i] = j;
                if (lru) atomicMax(&sm.b_stamp[j], t);
                intra = 1;
            }
        }
    }
    const int n_intra = __syncthreads_count(intra);
    if (i == 0) {
        st->count = count0 + n_free;
        if (policy == PROX_FIFO) st->fifo_head = (st->fifo_head + n_evict) % C;
        st->clock = clock0 + B;
        st->n_miss = total_miss;
        st->queries += B;
        st->hits += B - total_miss;
        st->misses += total_miss;
        st->intra_hits += n_intra;
        st->evictions += n_evict;
        st->parallel_replays += 1;
    }
    return true;
}

// The whole replay, for a block of 1024 threads (sm: the block's ResolveSmem).
__device__ void resolve_block(ResolveSmem &sm, DevState *st, int B, long long C, double tau, int policy, u64 *stamp,
                              const int32_t *risk_slot, const u64 *risk_stamp,
                              const double *g_safe_min, const int32_t *g_safe_arg,
                              const double *cand_d, const int32_t *cand_code,
                              const int32_t *n_cand, uint8_t *out_hit, int32_t *src, int32_t *src_kind,
                              int32_t *ins_slot, int32_t *evt_slot, float *evt_dist, int32_t *miss_list,
                              int32_t *miss_rank, bool allow_parallel) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int R = st->n_risk;
    const long long count0 = st->count, clock0 = st->clock;
    ResolveOut o{out_hit, src, src_kind, evt_slot, miss_list, miss_rank, evt_dist};

    // ---- load and classify
    int n_plain = 0, n_ent = 0, n_settled = 0;
    {
        const int i = tid;
        int n = 0, kind = 0;                               // 1 settled, 2 plain miss, 3 entangled
        double sd = INFINITY;
        int sa = -1;
        bool safe_hit = false;
        if (i < B) {
            n = n_cand[i];
            sd = g_safe_min[i];
            sa = g_safe_arg[i];
            sm.safe_min[i] = sd;
            sm.safe_arg[i] = sa;
            sm.b_slot[i] = -1;
            sm.b_stamp[i] = 0;
            safe_hit = sa >= 0 && sd <= tau;
            kind = n > 0 ? 3 : (safe_hit ? 1 : 2);
        }
        if (i < R) {
            sm.r_slot[i] = risk_slot[i];
            sm.r_stamp[i] = risk_stamp[i];
            sm.r_alive[i] = 1;
            sm.r_touched[i] = 0;
        }
        if (i < kMaxBatch) { sm.ncand[i] = n; sm.kind[i] = (unsigned char)kind; sm.head[i] = 0; }
        // exclusive prefix sum of the list lengths: where each list sits in the shared copy
        int x = n;
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, x, m);
            if (lane >= m) x += y;
        }
        if (lane == 31) sm.warp_tot[0][warp] = x;
        __syncthreads();
        if (warp == 0) {
            int w = sm.warp_tot[0][lane];
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, w, m);
                if (lane >= m) w += y;
            }
            sm.warp_tot[0][lane] = w;
        }
        __syncthreads();
        const int incl_n = x + (warp > 0 ? sm.warp_tot[0][warp - 1] : 0);
        if (i < kMaxBatch) sm.off[i] = incl_n - n;
        if (i == kMaxBatch - 1) sm.off[kMaxBatch] = incl_n;
        __syncthreads();
        for (int row = warp; row < B; row += 32) {
            const int off = sm.off[row], nn = sm.ncand[row];
            if (off + nn <= kCsrCap)
                for (int e = lane; e < nn; e += 32) {
                    sm.csr_d[off + e] = cand_d[(size_t)row * (2 * kMaxBatch) + e];
                    sm.csr_code[off + e] = cand_code[(size_t)row * (2 * kMaxBatch) + e];
                }
        }
        __syncthreads();

        // Most queries with a listed key can still be decided without the others.  A listed query of
        // the batch that is known to hit was never inserted: it cannot be anyone's key, so it drops
        // off the front of the lists; and when the nearest safe key is strictly nearer than the first
        // listed key that could still be resident, the query hits that safe key whatever happens to
        // the listed ones.  A few rounds, each one settling what the round before made decidable.
        for (int round = 0; round < 4; ++round) {
            bool changed = false;
            if (i < B && kind == 3) {
                const int off = sm.off[i];
                const bool in_smem = off + n <= kCsrCap;
                const int *lc = in_smem ? sm.csr_code + off : cand_code + (size_t)i * (2 * kMaxBatch);
                const double *ld = in_smem ? sm.csr_d + off : cand_d + (size_t)i * (2 * kMaxBatch);
                int hd = sm.head[i];
                while (hd < n) {
                    const int code = lc[hd];
                    if (code >= kMaxBatch && sm.kind[code - kMaxBatch] == 1) ++hd;
                    else break;
                }
                sm.head[i] = hd;
                if (hd == n) { kind = safe_hit ? 1 : 2; changed = true; }
                else if (safe_hit && sd < ld[hd]) { kind = 1; changed = true; }
            }
            __syncthreads();                               // everyone has read the kinds of this pass
            if (changed) sm.kind[i] = (unsigned char)kind;
            if (!__syncthreads_or(changed ? 1 : 0)) break;
        }
        // a settled query hits its nearest safe key: safe keys are not evicted in this batch, and
        // touching one changes no eviction of this batch
        if (i < B && kind == 1) {
            out_hit[i] = 1;
            evt_slot[i] = sa;
            evt_dist[i] = (float)sd;
            miss_rank[i] = -1;
            src_kind[i] = 1; src[i] = sa;
            if (policy == PROX_LRU) atomicMax(&stamp[sa], (u64)(clock0 + i));     // the latest hit stays
        }

        // plain misses and entangled queries, each in index order
        int y2[2] = {kind == 2 ? 1 : 0, kind == 3 ? 1 : 0};
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                const int y = __shfl_up_sync(0xffffffffu, y2[c], m);
                if (lane >= m) y2[c] += y;
            }
        }
        if (lane == 31) { sm.warp_tot[1][warp] = y2[0]; sm.warp_tot[2][warp] = y2[1]; }
        __syncthreads();
        if (warp == 1 || warp == 2) {
            int w = sm.warp_tot[warp][lane];
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, w, m);
                if (lane >= m) w += y;
            }
            sm.warp_tot[warp][lane] = w;
        }
        __syncthreads();
        const int excl_plain = y2[0] + (warp > 0 ? sm.warp_tot[1][warp - 1] : 0) - (kind == 2 ? 1 : 0);
        const int excl_ent = y2[1] + (warp > 0 ? sm.warp_tot[2][warp - 1] : 0) - (kind == 3 ? 1 : 0);
        if (kind == 2) sm.plain_list[excl_plain] = i;
        if (kind == 3) { sm.ent_list[excl_ent] = i; sm.plain_before[excl_ent] = excl_plain; }
        n_plain = sm.warp_tot[1][31];
        n_ent = sm.warp_tot[2][31];
        n_settled = B - n_plain - n_ent;
        __syncthreads();
    }

    // ---- replay: all at once when many queries are entangled, else (or when that declines) in order by warp 0
    bool replayed = false;
    if (allow_parallel && n_ent >= kParallelMinEntangled)
        replayed = replay_parallel(sm, st, B, R, C, tau, policy, count0, clock0, cand_d, cand_code, stamp, o);
    if (!replayed && warp == 0) {
        ReplayState rs{count0, 0, 0, 0};
        int n_hit = n_settled, n_intra = 0, done_plain = 0;
        for (int k = 0; k < n_ent; ++k) {
            const int i = sm.ent_list[k];
            const int upto = sm.plain_before[k];
            if (upto > done_plain) {
                settle_misses(sm, rs, sm.plain_list, done_plain, upto, R, C, clock0, st, o);
                done_plain = upto;
            }
            const u64 t = (u64)(clock0 + i);
            const int n = sm.ncand[i], off = sm.off[i];
            const bool in_smem = (off + n <= kCsrCap);
            const double *ld = in_smem ? sm.csr_d + off : cand_d + (size_t)i * (2 * kMaxBatch);
            const int *lc = in_smem ? sm.csr_code + off : cand_code + (size_t)i * (2 * kMaxBatch);
            // the nearest entry of the sorted list that is still resident; among entries at exactly
            // the same distance the lowest slot
            double bd = INFINITY;
            int bslot = 0x7fffffff, bcode = -1;
            const int h0 = sm.head[i];
            {
                // common case, without a vote: the first listed entry is resident and no other entry is
                // exactly as near
                const int code = lc[h0];
                int slot;
                bool valid;
                if (code < kMaxBatch) { valid = sm.r_alive[code] != 0; slot = sm.r_slot[code]; }
                else { slot = sm.b_slot[code - kMaxBatch]; valid = slot >= 0; }
                const double d0 = ld[h0];
                if (valid && (h0 + 1 >= n || ld[h0 + 1] > d0)) { bd = d0; bslot = slot; bcode = code; }
            }
            for (int e0 = h0; e0 < n && bcode == -1; e0 += 32) {
                const int e = e0 + lane;
                int code = -1, slot = -1;
                bool valid = false;
                if (e < n) {
                    code = lc[e];
                    if (code < kMaxBatch) { valid = sm.r_alive[code] != 0; slot = sm.r_slot[code]; }
                    else { slot = sm.b_slot[code - kMaxBatch]; valid = slot >= 0; }
                }
                const unsigned mask = __ballot_sync(0xffffffffu, valid);
                if (mask == 0u) continue;
                const int first = __ffs(mask) - 1;
                bd = ld[e0 + first];
                bslot = __shfl_sync(0xffffffffu, slot, first);
                bcode = __shfl_sync(0xffffffffu, code, first);
                // entries at the same distance (in this group of 32 or beyond it)
                for (int f0 = e0; f0 < n; f0 += 32) {
                    const int f = f0 + lane;
                    bool same = false;
                    int fcode = -1, fslot = 0x7fffffff;
                    if (f < n && f > e0 + first && ld[f] == bd) {
                        fcode = lc[f];
                        if (fcode < kMaxBatch) { same = sm.r_alive[fcode] != 0; fslot = sm.r_slot[fcode]; }
                        else { fslot = sm.b_slot[fcode - kMaxBatch]; same = fslot >= 0; }
                    }
                    const bool past = f < n && ld[f] > bd;     // sorted: nothing equal follows
                    unsigned smask = __ballot_sync(0xffffffffu, same);
                    while (smask) {
                        const int l = __ffs(smask) - 1;
                        smask &= smask - 1;
                        const int os = __shfl_sync(0xffffffffu, fslot, l);
                        const int oc = __shfl_sync(0xffffffffu, fcode, l);
                        if (os < bslot) { bslot = os; bcode = oc; }
                    }
                    if (__any_sync(0xffffffffu, past)) break;
                }
            }
            {
                const double sd = sm.safe_min[i];
                const int sa = sm.safe_arg[i];
                if (sa >= 0 && sd <= tau && (sd < bd || (sd == bd && sa < bslot))) { bd = sd; bslot = sa; bcode = -2; }
            }
            if (bcode != -1) {                             // hit
                ++n_hit;
                if (lane == 0) {
                    out_hit[i] = 1;
                    evt_slot[i] = bslot;
                    evt_dist[i] = (float)bd;
                    miss_rank[i] = -1;
                    if (bcode == -2) {
                        src_kind[i] = 1; src[i] = bslot;
                        if (policy == PROX_LRU) atomicMax(&stamp[bslot], t);   // a later query may have touched it in the parallel pass
                    } else if (bcode < kMaxBatch) {
                        src_kind[i] = 1; src[i] = bslot;
                        if (policy == PROX_LRU) { sm.r_stamp[bcode] = t; sm.r_touched[bcode] = 1; }
                    } else {
                        src_kind[i] = 2; src[i] = bcode - kMaxBatch;
                        if (policy == PROX_LRU) sm.b_stamp[bcode - kMaxBatch] = t;
                    }
                }
                if (bcode >= kMaxBatch) ++n_intra;
                __syncwarp();
            } else {                                       // every key within tau has left: a miss after all
                if (lane == 0) sm.one[0] = i;
                __syncwarp();
                settle_misses(sm, rs, sm.one, 0, 1, R, C, clock0, st, o);
            }
        }
        if (n_plain > done_plain) settle_misses(sm, rs, sm.plain_list, done_plain, n_plain, R, C, clock0, st, o);
        if (lane == 0) {
            st->count = rs.cnt;
            if (policy == PROX_FIFO) st->fifo_head = (st->fifo_head + rs.n_evict) % C;   // the ring turns by one per eviction
            st->clock = clock0 + B;
            st->n_miss = rs.n_miss;
            st->queries += B;
            st->hits += n_hit;
            st->misses += rs.n_miss;
            st->intra_hits += n_intra;
            st->evictions += rs.n_evict;
        }
    }
    __syncthreads();

    // ---- write back stamps and the slots that entries of this batch own at batch end
    for (int r = tid; r < R; r += blockDim.x)
        if (sm.r_alive[r]) stamp[sm.r_slot[r]] = sm.r_stamp[r];
    for (int j = tid; j < B; j += blockDim.x) {
        const int s = sm.b_slot[j];
        ins_slot[j] = s;
        if (s >= 0) stamp[s] = sm.b_stamp[j];
    }
}

__global__ void __launch_bounds__(1024)
resolve_kernel(DevState *st, int B, long long C, double tau, int policy, u64 *stamp,
               const int32_t *__restrict__ risk_slot, const u64 *__restrict__ risk_stamp,
               const double *__restrict__ g_safe_min, const int32_t *__restrict__ g_safe_arg,
               const double *__restrict__ cand_d, const int32_t *__restrict__ cand_code,
               const int32_t *__restrict__ n_cand, uint8_t *out_hit, int32_t *src, int32_t *src_kind,
               int32_t *ins_slot, int32_t *evt_slot, float *evt_dist, int32_t *miss_list,
               int32_t *miss_rank, int allow_parallel) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ResolveSmem &sm = *reinterpret_cast<ResolveSmem *>(smem_raw);
    resolve_block(sm, st, B, C, tau, policy, stamp, risk_slot, risk_stamp, g_safe_min, g_safe_arg, cand_d, cand_code,
                  n_cand, out_hit, src, src_kind, ins_slot, evt_slot, evt_dist, miss_list, miss_rank, allow_parallel != 0);
}

// ------------------------------------------------------------------------------------------
// Small batches against a small cache (a query at a time, a few hundred keys): the work is a few
// microseconds, the cost is the chain of launches.  Two launches instead of five: all distances
// (every query against every stored key and every earlier query of the batch, fp64), then one
// block that picks the at-risk entries, finds the nearest safe key and the listed keys of every
// query, replays the batch and copies the stored lists of the hits.
// ------------------------------------------------------------------------------------------
constexpr int kSmallBatch = 4;                       // largest B of this path
constexpr int kSmallCapacity = 2048;                 // largest capacity of this path

template <bool IP>
__global__ void __launch_bounds__(256)
small_dist_kernel(const DevState *__restrict__ st, const float *__restrict__ keys, const float *__restrict__ queries,
                  int B, int d, int ld, double *__restrict__ d_all) {
    const long long count = st->count;
    const int lane = threadIdx.x & 31;
    const int warp = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, nwarps = (gridDim.x * blockDim.x) >> 5;
    for (long long col = warp; col < count + B; col += nwarps) {
        const float *x = col < count ? keys + (size_t)col * d : queries + (size_t)(col - count) * d;
        double acc[kSmallBatch];
#pragma unroll
        for (int i = 0; i < kSmallBatch; ++i) acc[i] = 0.0;
        for (int j = lane; j < d; j += 32) {
            const double xv = (double)x[j];
#pragma unroll
            for (int i = 0; i < kSmallBatch; ++i) {
                if (i < B) {
                    const double qv = (double)queries[(size_t)i * d + j];
                    if constexpr (IP) acc[i] = fma(-qv, xv, acc[i]);
                    else { const double df = qv - xv; acc[i] = fma(df, df, acc[i]); }
                }
            }
        }
#pragma unroll
        for (int i = 0; i < kSmallBatch; ++i) {
#pragma unroll
            for (int m = 16; m > 0; m >>= 1) acc[i] += __shfl_xor_sync(0xffffffffu, acc[i], m);
            if (lane == 0 && i < B) d_all[(size_t)i * ld + col] = acc[i];
        }
    }
}

__global__ void __launch_bounds__(1024)
small_resolve_kernel(DevState *st, int B, long long C, double tau, int policy, u64 *stamp, int32_t *risk_pos,
                     int32_t *risk_slot, u64 *risk_stamp, const double *__restrict__ d_all, int ld, double *safe_min,
                     int32_t *safe_arg, double *cand_d, int32_t *cand_code, int32_t *n_cand, uint8_t *out_hit,
                     int32_t *src, int32_t *src_kind, int32_t *ins_slot, int32_t *evt_slot, float *evt_dist,
                     int32_t *miss_list, int32_t *miss_rank, int k, const int32_t *__restrict__ val_ids,
                     const float *__restrict__ val_dists, int64_t *out_ids, float *out_dists) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    ResolveSmem &sm = *reinterpret_cast<ResolveSmem *>(smem_raw);
    __shared__ unsigned hist[256];
    __shared__ u64 s_key[1024];
    __shared__ int s_val[1024];
    __shared__ u64 s_prefix, s_mask;
    __shared__ int s_remaining, s_n;
    __shared__ double s_d[4 * kSmallBatch];            // at most R + B - 1 <= 2 B - 1 listed keys per query
    __shared__ int s_code[4 * kSmallBatch];
    __shared__ double w_d[32];
    __shared__ int w_s[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    // ---- the at-risk entries of this batch
    const int prev = st->n_risk;
    for (int r = tid; r < prev; r += blockDim.x) risk_pos[risk_slot[r]] = -1;
    const long long count = st->count, clock = st->clock;
    __syncthreads();
    const int R = risk_count(count, B, C);
    if (R > 0) {
        const int found = select_smallest(stamp, nullptr, count, R, clock, hist, s_key, s_val, &s_prefix, &s_mask,
                                          &s_remaining, &s_n);
        if (found != R) {                    // stamps must be unique; anything else is a broken state
            if (tid == 0) { atomicCAS(&st->error, 0, PROX_ERR_INTERNAL); st->n_risk = 0; }
            return;
        }
        publish_risk_list(st, R, s_key, s_val, risk_pos, risk_slot, risk_stamp);
    } else if (tid == 0) {
        st->n_risk = 0;
    }
    __syncthreads();

    // ---- per query: the nearest safe key, and the at-risk and in-batch keys within tau, nearest first
    for (int i = 0; i < B; ++i) {
        const double *row = d_all + (size_t)i * ld;
        double bd = INFINITY;
        int bs = 0x7fffffff;
        for (long long c = tid; c < count; c += blockDim.x) {
            if (risk_pos[c] >= 0) continue;
            const double v = row[c];
            if (v < bd || (v == bd && (int)c < bs)) { bd = v; bs = (int)c; }
        }
#pragma unroll
        for (int m = 1; m < 32; m <<= 1) {
            const double od = __shfl_xor_sync(0xffffffffu, bd, m);
            const int os = __shfl_xor_sync(0xffffffffu, bs, m);
            if (od < bd || (od == bd && os < bs)) { bd = od; bs = os; }
        }
        if (lane == 0) { w_d[warp] = bd; w_s[warp] = bs; }
        if (tid == 0) s_n = 0;
        __syncthreads();
        if (warp == 0) {
            bd = w_d[lane]; bs = w_s[lane];
#pragma unroll
            for (int m = 1; m < 32; m <<= 1) {
                const double od = __shfl_xor_sync(0xffffffffu, bd, m);
                const int os = __shfl_xor_sync(0xffffffffu, bs, m);
                if (od < bd || (od == bd && os < bs)) { bd = od; bs = os; }
            }
            if (lane == 0) { safe_min[i] = bd; safe_arg[i] = bs == 0x7fffffff ? -1 : bs; }
        }
        for (int e = tid; e < R + i; e += blockDim.x) {
            const double v = e < R ? row[risk_slot[e]] : row[count + (e - R)];
            if (v <= tau) {
                const int pos = atomicAdd(&s_n, 1);
                s_d[pos] = v;
                s_code[pos] = e < R ? e : kMaxBatch + (e - R);
            }
        }
        __syncthreads();
        const int n = s_n;
        if (n > 1) {
            int n2 = 2;
            while (n2 < n) n2 <<= 1;
            for (int e = n + tid; e < n2; e += blockDim.x) { s_d[e] = INFINITY; s_code[e] = 0x7fffffff; }
            block_sort_asc(s_d, s_code, n2);
        }
        for (int e = tid; e < n; e += blockDim.x) {
            cand_d[(size_t)i * (2 * kMaxBatch) + e] = s_d[e];
            cand_code[(size_t)i * (2 * kMaxBatch) + e] = s_code[e];
        }
        if (tid == 0) n_cand[i] = n;
        __syncthreads();
    }

    // ---- replay, then the stored lists of the hits on keys that were there before the batch
    resolve_block(sm, st, B, C, tau, policy, stamp, risk_slot, risk_stamp, safe_min, safe_arg, cand_d, cand_code, n_cand,
                  out_hit, src, src_kind, ins_slot, evt_slot, evt_dist, miss_list, miss_rank, false);
    if (out_ids != nullptr) {
        __syncthreads();
        for (int i = 0; i < B; ++i) {
            if (src_kind[i] != 1) continue;
            const int sl = src[i];
            for (int r = tid; r < k; r += blockDim.x) {
                out_ids[(size_t)i * k + r] = (int64_t)val_ids[(size_t)sl * k + r];
                out_dists[(size_t)i * k + r] = val_dists[(size_t)sl * k + r];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Value-slot traffic.
// ------------------------------------------------------------------------------------------
// Hits on a key that was resident before the batch: copy its stored list (the hit branch of Algorithm 1).
// Runs before any slot is overwritten by this batch.
__global__ void gather_hits_kernel(int B, int k, const int32_t *__restrict__ src,
                                   const int32_t *__restrict__ src_kind,
                                   const int32_t *__restrict__ val_ids,
                                   const float *__restrict__ val_dists, int64_t *out_ids,
                                   float *out_dists) {
    const int i = blockIdx.x;
    if (i >= B || src_kind[i] != 1) return;
    const int s = src[i];
    for (int r = threadIdx.x; r < k; r += blockDim.x) {
        out_ids[(size_t)i * k + r] = (int64_t)val_ids[(size_t)s * k + r];
        out_dists[(size_t)i * k + r] = val_dists[(size_t)s * k + r];
    }
}

// Misses return their fresh list (the end of Algorithm 1); hits on a key inserted earlier in the batch return
// that query's list; entries that own a slot at batch end are written (the insertion of Algorithm 1).
__global__ void scatter_kernel(int B, int d, int k, int k_out, int with_values, const float *__restrict__ queries,
                               const int32_t *__restrict__ src, const int32_t *__restrict__ src_kind,
                               const int32_t *__restrict__ ins_slot,
                               const int32_t *__restrict__ miss_rank,
                               const int32_t *__restrict__ res_ids,
                               const double *__restrict__ res_dists, float *keys, int32_t *val_ids,
                               float *val_dists, int64_t *out_ids, float *out_dists, __nv_bfloat16 *keys_b,
                               float *kh, DevState *st) {
    __shared__ float red[2][4];
    const int i = blockIdx.x;
    if (i >= B) return;
    const int kind = src_kind[i];
    const int owner = (kind == 0) ? i : (kind == 2 ? src[i] : -1);
    const int m = (owner >= 0) ? miss_rank[owner] : -1;
    // a miss returns the k_out nearest of the k rows it fetched; with re-ranking (k > k_out) a hit
    // on a key of this batch was answered by the re-ranking kernel
    if (with_values && m >= 0 && (kind == 0 || k == k_out)) {
        for (int r = threadIdx.x; r < k_out; r += blockDim.x) {
            out_ids[(size_t)i * k_out + r] = (int64_t)res_ids[(size_t)m * k + r];
            out_dists[(size_t)i * k_out + r] = (float)res_dists[(size_t)m * k + r];
        }
    }
    const int slot = ins_slot[i];
    if (slot >= 0) {
        float nn = 0.f, ee = 0.f;
        for (int j = threadIdx.x; j < d; j += blockDim.x) {
            const float v = queries[(size_t)i * d + j];
            keys[(size_t)slot * d + j] = v;
            if (keys_b) {                                 // bf16 copy for the coarse probe
                const __nv_bfloat16 b = __float2bfloat16_rn(v);
                const float f = __bfloat162float(b);
                keys_b[(size_t)slot * d + j] = b;
                nn += f * f;
                ee += (v - f) * (v - f);
            }
        }
        for (int r = threadIdx.x; r < k; r += blockDim.x) {
            val_ids[(size_t)slot * k + r] = with_values ? res_ids[(size_t)m * k + r] : -1;
            val_dists[(size_t)slot * k + r] = with_values ? (float)res_dists[(size_t)m * k + r] : 0.f;
        }
        if (keys_b) {
#pragma unroll
            for (int sft = 16; sft > 0; sft >>= 1) {
                nn += __shfl_xor_sync(0xffffffffu, nn, sft);
                ee += __shfl_xor_sync(0xffffffffu, ee, sft);
            }
            if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = nn; red[1][threadIdx.x >> 5] = ee; }
            __syncthreads();
            if (threadIdx.x == 0) {
                const float n2 = red[0][0] + red[0][1] + red[0][2] + red[0][3];
                const float e2 = red[1][0] + red[1][1] + red[1][2] + red[1][3];
                kh[slot] = 0.5f * n2;
                atomicMax(reinterpret_cast<int *>(&st->ke_max), __float_as_int(sqrtf(e2) * 1.0001f));
                atomicMax(reinterpret_cast<int *>(&st->kn_max), __float_as_int(sqrtf(n2) * 1.0001f));
            }
        }
    }
}

__global__ void copy_probe_outputs_kernel(int B, const int32_t *__restrict__ evt_slot,
                                          const float *__restrict__ evt_dist, int32_t *out_slot,
                                          float *out_min_dist) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= B) return;
    if (out_slot) out_slot[i] = evt_slot[i];
    if (out_min_dist) out_min_dist[i] = evt_dist[i];
}

__global__ void reset_kernel(DevState *st, int32_t *risk_pos, long long C, long long n_loaded, float *kh) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < C) {
        risk_pos[i] = -1;
        if (kh) kh[i] = INFINITY;                         // an empty slot can never pass the coarse probe
    }
    if (i == 0) {
        const float e_max = st->e_max, xn_max = st->xn_max;
        const int err = st->error;
        *st = DevState{};
        st->e_max = e_max;
        st->xn_max = xn_max;
        st->error = err;
        st->count = n_loaded;
        st->clock = n_loaded;
    }
}

__global__ void cache_load_kernel(long long n, int d, int k, const float *__restrict__ src, float *keys,
                                  int32_t *val_ids, float *val_dists, u64 *stamp, __nv_bfloat16 *keys_b, float *kh,
                                  DevState *st) {
    __shared__ float red[2][4];
    const long long s = blockIdx.x;
    if (s >= n) return;
    float nn = 0.f, ee = 0.f;
    for (int j = threadIdx.x; j < d; j += blockDim.x) {
        const float v = src[(size_t)s * d + j];
        keys[(size_t)s * d + j] = v;
        if (keys_b) {
            const __nv_bfloat16 b = __float2bfloat16_rn(v);
            const float f = __bfloat162float(b);
            keys_b[(size_t)s * d + j] = b;
            nn += f * f;
            ee += (v - f) * (v - f);
        }
    }
    if (keys_b) {
#pragma unroll
        for (int sft = 16; sft > 0; sft >>= 1) {
            nn += __shfl_xor_sync(0xffffffffu, nn, sft);
            ee += __shfl_xor_sync(0xffffffffu, ee, sft);
        }
        if ((threadIdx.x & 31) == 0) { red[0][threadIdx.x >> 5] = nn; red[1][threadIdx.x >> 5] = ee; }
        __syncthreads();
        if (threadIdx.x == 0) {
            const float n2 = red[0][0] + red[0][1] + red[0][2] + red[0][3];
            const float e2 = red[1][0] + red[1][1] + red[1][2] + red[1][3];
            kh[s] = 0.5f * n2;
            atomicMax(reinterpret_cast<int *>(&st->ke_max), __float_as_int(sqrtf(e2) * 1.0001f));
            atomicMax(reinterpret_cast<int *>(&st->kn_max), __float_as_int(sqrtf(n2) * 1.0001f));
        }
    }
    for (int r = threadIdx.x; r < k; r += blockDim.x) {
        val_ids[(size_t)s * k + r] = -1;
        val_dists[(size_t)s * k + r] = 0.f;
    }
    if (threadIdx.x == 0) stamp[s] = (u64)s;
}

// ------------------------------------------------------------------------------------------
// Launchers
// ------------------------------------------------------------------------------------------
// Columns per tile of the fp64 probe: narrow tiles when wide ones would not give every SM two blocks.
static int probe_cols(const prox_handle *h, int B) {
    const long long wide = (h->C + B + kProbeColsWide - 1) / kProbeColsWide;
    const int qtiles = (B + PQ - 1) / PQ;
    if (wide * qtiles >= 2LL * h->num_sms) return kProbeColsWide;
    // fewer blocks than SMs even with narrow tiles (a small batch against a small cache): halve the tiles again
    const long long narrow = (h->C + B + kProbeColsNarrow - 1) / kProbeColsNarrow;
    return narrow * qtiles < h->num_sms ? kProbeColsTiny : kProbeColsNarrow;
}

static int probe_splits(const prox_handle *h, int B) {
    const int PC = probe_cols(h, B);
    const long long ntiles = (h->C + B + PC - 1) / PC;
    const int qtiles = (B + PQ - 1) / PQ;
    long long want = (4LL * h->num_sms + qtiles - 1) / qtiles;     // about four blocks per SM
    if (want > ntiles) want = ntiles;
    if (want > kProbeSplitMax) want = kProbeSplitMax;
    if (want < 1) want = 1;
    return (int)want;
}

// dst row = src row / |src row| (norm and quotient in fp64, rounded to fp32 once); one warp per row.
// dst may be src.
__global__ void __launch_bounds__(256)
normalize_rows_kernel(const float *src, float *dst, long long n, int d) {
    const long long r = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (r >= n) return;
    const float *x = src + (size_t)r * d;
    double acc = 0.0;
    for (int j = lane; j < d; j += 32) acc += (double)x[j] * (double)x[j];
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
    const double nrm = sqrt(acc);
    float *y = dst + (size_t)r * d;
    for (int j = lane; j < d; j += 32) y[j] = (float)((double)x[j] / nrm);
}

__global__ void scale_kernel(float *v, long long n, float f) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) v[i] *= f;
}

void launch_normalize_rows(const float *src, float *dst, long long n, int d, cudaStream_t s) {
    normalize_rows_kernel<<<(unsigned)((n + 7) / 8), 256, 0, s>>>(src, dst, n, d);
}

void launch_scale(float *v, long long n, float f, cudaStream_t s) {
    scale_kernel<<<(unsigned)((n + 255) / 256), 256, 0, s>>>(v, n, f);
}

void launch_risk_select(prox_handle *h, int B, cudaStream_t s) {
    if (h->policy == PROX_FIFO) {
        risk_ring_kernel<<<1, 1024, 0, s>>>(h->st, h->stamp, h->risk_pos, h->risk_slot, h->risk_stamp, B, (long long)h->C);
        h->launches++;
        return;
    }
    // one block reads a small cache faster than four launches do
    if (h->C <= (1 << 16)) {
        risk_select_kernel<<<1, 1024, 0, s>>>(h->st, h->stamp, h->risk_pos, h->risk_slot, h->risk_stamp, B,
                                              (long long)h->C);
        h->launches++;
        return;
    }
    // the work area borrows the candidate table of the resolve, which is filled later in the batch
    static_assert(sizeof(RiskWork) <= sizeof(double) * (size_t)kMaxBatch * 2 * kMaxBatch, "work area too large");
    RiskWork *w = reinterpret_cast<RiskWork *>(h->cand_d);
    cudaMemsetAsync(w->hist, 0, sizeof(w->hist), s);
    const int grid = h->num_sms * 8;
    risk_hist_kernel<<<grid, 256, 0, s>>>(h->st, h->stamp, h->risk_pos, h->risk_slot, w, B, (long long)h->C);
    risk_pick_kernel<<<1, 1024, 0, s>>>(h->st, w, B, (long long)h->C);
    risk_collect_kernel<<<grid, 256, 0, s>>>(h->st, h->stamp, w, B, (long long)h->C);
    risk_finish_kernel<<<1, 1024, 0, s>>>(h->st, w, h->risk_pos, h->risk_slot, h->risk_stamp, B, (long long)h->C);
    h->launches += 4;
}

void launch_probe(prox_handle *h, const float *q, int B, int mode, cudaStream_t s) {
    int splits = probe_splits(h, B);
    const int PC = probe_cols(h, B);
    if (mode == 1 || mode == 4) {                         // at most 2 * kMaxBatch columns
        const int tiles = (2 * B + PC - 1) / PC;
        if (splits > tiles) splits = tiles;
    }
    dim3 grid((B + PQ - 1) / PQ, splits);
    auto kern = PC == kProbeColsTiny     ? (metric_is_ip(h) ? probe_kernel<kProbeColsTiny, 64, true> : probe_kernel<kProbeColsTiny, 64, false>)
                : PC == kProbeColsNarrow ? (metric_is_ip(h) ? probe_kernel<kProbeColsNarrow, 64, true> : probe_kernel<kProbeColsNarrow, 64, false>)
                                         : (metric_is_ip(h) ? probe_kernel<kProbeColsWide, 32, true> : probe_kernel<kProbeColsWide, 32, false>);
    kern<<<grid, 256, 0, s>>>(h->st, h->keys, q, h->risk_pos, B, h->d, h->part_min, h->part_arg, h->d_risk, h->d_intra, mode,
                              h->risk_slot, h->pfail_list);
    h->launches++;
}

void launch_build_candidates(prox_handle *h, int B, int splits, int lists_ready, cudaStream_t s) {
    build_candidates_kernel<<<B, 128, 0, s>>>(h->st, B, splits < 0 ? probe_splits(h, B) : splits, (double)h->tau, h->part_min,
                                              h->part_arg, h->d_risk, h->d_intra, h->safe_min,
                                              h->safe_arg, h->cand_d, h->cand_code, h->n_cand,
                                              h->probe_tc ? h->use_partial : nullptr, lists_ready);
    h->launches++;
}

// Kernel attributes belong to a device: set when a handle is created there, not once per process.
void set_cache_kernel_attributes() {
    cudaFuncSetAttribute(resolve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ResolveSmem));
    cudaFuncSetAttribute(small_resolve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(ResolveSmem));
}

void launch_resolve(prox_handle *h, int B, uint8_t *out_hit, cudaStream_t s) {
    resolve_kernel<<<1, 1024, sizeof(ResolveSmem), s>>>(
        h->st, B, (long long)h->C, (double)h->tau, h->policy, h->stamp, h->risk_slot, h->risk_stamp,
        h->safe_min, h->safe_arg, h->cand_d, h->cand_code, h->n_cand, out_hit, h->src, h->src_kind,
        h->ins_slot, h->evt_slot, h->evt_dist, h->miss_list, h->miss_rank,
        h->scan_mode != PROX_SCAN_CUDA_CORE ? 1 : 0);      // the cross-check mode replays in query order
    h->launches++;
}

// B and capacity small enough for the two-launch path (the handle's own distance; any policy).
bool small_lookup_fits(const prox_handle *h, int B) { return B <= kSmallBatch && h->C <= kSmallCapacity && h->lsh_L < 0; }

// Probe, at-risk selection, candidates, replay and (with out_ids) the gather of the hits' stored lists.
void launch_small_lookup(prox_handle *h, const float *q, int B, uint8_t *out_hit, int64_t *out_ids, float *out_dists,
                         cudaStream_t s) {
    const int ld = (int)h->C + B;
    const int blocks = (ld + 7) / 8;
    if (metric_is_ip(h)) small_dist_kernel<true><<<blocks, 256, 0, s>>>(h->st, h->keys, q, B, h->d, ld, h->d_risk);
    else small_dist_kernel<false><<<blocks, 256, 0, s>>>(h->st, h->keys, q, B, h->d, ld, h->d_risk);
    small_resolve_kernel<<<1, 1024, sizeof(ResolveSmem), s>>>(
        h->st, B, (long long)h->C, (double)h->tau, h->policy, h->stamp, h->risk_pos, h->risk_slot, h->risk_stamp, h->d_risk,
        ld, h->safe_min, h->safe_arg, h->cand_d, h->cand_code, h->n_cand, out_hit, h->src, h->src_kind, h->ins_slot,
        h->evt_slot, h->evt_dist, h->miss_list, h->miss_rank, h->k, h->val_ids, h->val_dists, out_ids, out_dists);
    h->launches += 2;
}

void launch_gather_hits(prox_handle *h, int B, int64_t *out_ids, float *out_dists, cudaStream_t s) {
    gather_hits_kernel<<<B, 64, 0, s>>>(B, h->k, h->src, h->src_kind, h->val_ids, h->val_dists, out_ids,
                                        out_dists);
    h->launches++;
}

void launch_scatter(prox_handle *h, const float *q, int B, int64_t *out_ids, float *out_dists,
                    int with_values, cudaStream_t s) {
    scatter_kernel<<<B, 128, 0, s>>>(B, h->d, h->k, h->k_out, with_values, q, h->src, h->src_kind, h->ins_slot,
                                     h->miss_rank, h->res_ids, h->res_dists, h->keys, h->val_ids,
                                     h->val_dists, out_ids, out_dists, h->key_copies ? h->keys_b : nullptr, h->kh,
                                     h->st);
    h->launches++;
}

void launch_probe_outputs(prox_handle *h, int B, int32_t *out_slot, float *out_min_dist, cudaStream_t s) {
    copy_probe_outputs_kernel<<<(B + 255) / 256, 256, 0, s>>>(B, h->evt_slot, h->evt_dist, out_slot,
                                                             out_min_dist);
    h->launches++;
}

void launch_reset(prox_handle *h, cudaStream_t s) {
    const long long C = h->C;
    reset_kernel<<<(unsigned)((C + 255) / 256), 256, 0, s>>>(h->st, h->risk_pos, C, 0, h->key_copies ? h->kh : nullptr);
    h->launches++;
}

void launch_cache_load(prox_handle *h, const float *keys, int64_t n, cudaStream_t s) {
    const long long C = h->C;
    reset_kernel<<<(unsigned)((C + 255) / 256), 256, 0, s>>>(h->st, h->risk_pos, C, (long long)n, h->key_copies ? h->kh : nullptr);
    h->launches++;
    if (n > 0) {
        cache_load_kernel<<<(unsigned)n, 128, 0, s>>>((long long)n, h->d, h->k, keys, h->keys, h->val_ids,
                                                      h->val_dists, h->stamp, h->key_copies ? h->keys_b : nullptr,
                                                      h->kh, h->st);
        h->launches++;
    }
}

}  // namespace prox
