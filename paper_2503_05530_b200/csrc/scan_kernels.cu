// Miss path: exact k nearest corpus rows for the queries that missed (the database call of Algorithm 1,
// with an exact flat index as in Section 4.2.1).
//
// Route to the exact answer:
//   1. coarse scores  s(q, x) = bf16(q).bf16(x) - |bf16(x)|^2 / 2   for every corpus row, so that
//      |bf16(q) - bf16(x)|^2 = |bf16(q)|^2 - 2 s; the k' rows with the largest s are kept per
//      query (this file: the CUDA-core version of that scan; scan_tcgen05.cu: tensor cores);
//   2. the k' candidates are measured exactly, sum_j (q_j - x_j)^2 in fp64 over the fp32 rows,
//      and sorted by (distance, row id): the first k are the answer if the certificate holds;
//   3. certificate: with a = |q - bf16(q)| and e >= |x - bf16(x)| for every row, a row outside
//      the candidate set has coarse distance >= c' (the k'-th best), hence true distance
//      >= (sqrt(c') - a - e)^2.  If the exact k-th candidate distance is below that bound, no
//      outside row can belong to the top k;
//   4. otherwise (rare) the query takes an exact fp32 pass over the whole corpus that collects
//      every row within the k-th candidate distance (plus the fp32 rounding margin), and those
//      rows are measured in fp64 like the candidates.
#include <cfloat>
#include <cmath>

#include "prox_internal.h"
#include "topk_device.cuh"

namespace prox {


// ------------------------------------------------------------------------------------------
// Create time: bf16 copy (round to nearest even), half squared norms of the rounded rows and
// the largest rounding error norm.  One warp per row.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
convert_corpus_kernel(const float *__restrict__ x, long long N, int d, __nv_bfloat16 *__restrict__ xb,
                      float *__restrict__ xh, DevState *st, int ip) {
    const int lane = threadIdx.x & 31;
    const long long warp = ((long long)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    float emax = 0.f, nmax = 0.f;
    for (long long r = warp; r < N; r += nwarps) {
        const float *src = x + (size_t)r * d;
        __nv_bfloat16 *dst = xb + (size_t)r * d;
        float nn = 0.f, ee = 0.f;
        for (int j = lane * 4; j < d; j += 128) {
            const float4 v = *reinterpret_cast<const float4 *>(src + j);
            const __nv_bfloat16 b0 = __float2bfloat16_rn(v.x), b1 = __float2bfloat16_rn(v.y),
                                b2 = __float2bfloat16_rn(v.z), b3 = __float2bfloat16_rn(v.w);
            const float f0 = __bfloat162float(b0), f1 = __bfloat162float(b1), f2 = __bfloat162float(b2),
                        f3 = __bfloat162float(b3);
            nn += f0 * f0 + f1 * f1 + f2 * f2 + f3 * f3;
            ee += (v.x - f0) * (v.x - f0) + (v.y - f1) * (v.y - f1) + (v.z - f2) * (v.z - f2) +
                  (v.w - f3) * (v.w - f3);
            __nv_bfloat162 p0, p1;
            p0.x = b0; p0.y = b1; p1.x = b2; p1.y = b3;
            *reinterpret_cast<__nv_bfloat162 *>(dst + j) = p0;
            *reinterpret_cast<__nv_bfloat162 *>(dst + j + 2) = p1;
        }
#pragma unroll
        for (int m = 16; m > 0; m >>= 1) {
            nn += __shfl_xor_sync(0xffffffffu, nn, m);
            ee += __shfl_xor_sync(0xffffffffu, ee, m);
        }
        if (lane == 0) xh[r] = ip ? 0.f : 0.5f * nn;      // inner product: the coarse score is the product alone
        emax = fmaxf(emax, ee);
        nmax = fmaxf(nmax, nn);
    }
    if (lane == 0) {                                       // positive floats order as ints
        atomicMax(reinterpret_cast<int *>(&st->e_max), __float_as_int(sqrtf(emax) * 1.0001f));
        atomicMax(reinterpret_cast<int *>(&st->xn_max), __float_as_int(sqrtf(nmax) * 1.0001f));
    }
}

// ------------------------------------------------------------------------------------------
// Per batch: bf16 copies of the miss queries in miss order, their norms and rounding errors;
// resets of the per-batch scan state.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(128)
prep_miss_kernel(DevState *st, const float *__restrict__ queries, int B, int d,
                 const int32_t *__restrict__ miss_list, __nv_bfloat16 *qb, float *qbn, float *qerr,
                 uint32_t *thr_g, int32_t *coll_n, uint32_t *top1, int n_blocks) {
    __shared__ float red[2][4];
    const int m = blockIdx.x, tid = threadIdx.x;
    const int n_miss = st->n_miss;
    for (int i = tid; i < n_blocks; i += blockDim.x) top1[(size_t)m * n_blocks + i] = 0u;
    if (m == 0) {
        for (int i = tid; i < kMaxBatch; i += blockDim.x) {
            thr_g[i] = f2o(-INFINITY);
            coll_n[i] = 0;
        }
        if (tid == 0) {
            st->n_fail = 0;
            st->n_over = 0;
            if (n_miss > 0) st->scan_batches++;
        }
    }
    if (m >= n_miss) {
        for (int j = tid; j < d; j += blockDim.x) qb[(size_t)m * d + j] = __float2bfloat16_rn(0.f);
        return;
    }
    const float *src = queries + (size_t)miss_list[m] * d;
    float nn = 0.f, ee = 0.f;
    for (int j = tid; j < d; j += blockDim.x) {
        const float v = src[j];
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        const float f = __bfloat162float(b);
        qb[(size_t)m * d + j] = b;
        nn += f * f;
        ee += (v - f) * (v - f);
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        nn += __shfl_xor_sync(0xffffffffu, nn, s);
        ee += __shfl_xor_sync(0xffffffffu, ee, s);
    }
    if ((tid & 31) == 0) { red[0][tid >> 5] = nn; red[1][tid >> 5] = ee; }
    __syncthreads();
    if (tid == 0) {
        qbn[m] = red[0][0] + red[0][1] + red[0][2] + red[0][3];
        qerr[m] = sqrtf(red[1][0] + red[1][1] + red[1][2] + red[1][3]) * 1.0001f;
    }
}

// ------------------------------------------------------------------------------------------
// Candidate buffers.  Each scanning block owns, per query of the pass, kBufCap entries in
// global memory.  A score enters the buffer if it beats the query's threshold; when a
// buffer could overflow during the next tile, a warp sorts it, keeps the best k' and raises
// the threshold to the k'-th score.  Thresholds are shared between blocks through thr_g (a
// block's k'-th best is a lower bound of the global k'-th best).
// ------------------------------------------------------------------------------------------
// CUDA-core scan of one pass (up to kScanQ miss queries): tile = 128 rows x 64 queries,
// d in chunks of 32, fp32 accumulation of bf16 products.
__global__ void __launch_bounds__(256)
scan_cc_kernel(const DevState *__restrict__ st, const __nv_bfloat16 *__restrict__ xb,
               const float *__restrict__ xh, const __nv_bfloat16 *__restrict__ qb, long long N, int d,
               int pass, int kp, uint32_t *thr_g, uint32_t *top1, u64 *buf, int32_t *buf_cnt) {
    __shared__ float xs[kTileRows][33];
    __shared__ float qs[64][33];
    __shared__ float thr[kScanQ];
    __shared__ int cnt[kScanQ];
    const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4, warp = tid >> 5;
    const int q0 = pass * kScanQ;
    int nq = st->n_miss - q0;
    if (nq > kScanQ) nq = kScanQ;
    if (nq <= 0) return;
    thr_g += q0;
    top1 += (size_t)q0 * gridDim.x;
    u64 *mybuf = buf + (size_t)blockIdx.x * kScanQ * kBufCap;
    for (int q = tid; q < kScanQ; q += blockDim.x) { thr[q] = -INFINITY; cnt[q] = 0; }
    __syncthreads();

    const long long ntiles = (N + kTileRows - 1) / kTileRows;
    for (long long tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        const long long row0 = tile * kTileRows;
        for (int q = tid; q < nq; q += blockDim.x) thr[q] = fmaxf(thr[q], o2f(thr_g[q]));
        for (int qg = 0; qg < nq; qg += 64) {
            float acc[8][4];
#pragma unroll
            for (int a = 0; a < 8; ++a)
#pragma unroll
                for (int b = 0; b < 4; ++b) acc[a][b] = 0.f;
            for (int kc = 0; kc < d; kc += 32) {
                __syncthreads();
#pragma unroll
                for (int it = 0; it < 16; ++it) {
                    const int idx = it * 256 + tid, r = idx >> 5, c = idx & 31;
                    const long long row = row0 + r;
                    xs[r][c] = (row < N && kc + c < d) ? __bfloat162float(xb[(size_t)row * d + kc + c]) : 0.f;
                }
#pragma unroll
                for (int it = 0; it < 8; ++it) {
                    const int idx = it * 256 + tid, r = idx >> 5, c = idx & 31;
                    const int q = qg + r;
                    qs[r][c] = (q < nq && kc + c < d) ? __bfloat162float(qb[(size_t)(q0 + q) * d + kc + c]) : 0.f;
                }
                __syncthreads();
#pragma unroll 4
                for (int j = 0; j < 32; ++j) {
                    float xv[8], qv[4];
#pragma unroll
                    for (int a = 0; a < 8; ++a) xv[a] = xs[ty + 16 * a][j];
#pragma unroll
                    for (int b = 0; b < 4; ++b) qv[b] = qs[tx + 16 * b][j];
#pragma unroll
                    for (int a = 0; a < 8; ++a)
#pragma unroll
                        for (int b = 0; b < 4; ++b) acc[a][b] = fmaf(xv[a], qv[b], acc[a][b]);
                }
            }
#pragma unroll
            for (int a = 0; a < 8; ++a) {
                const long long row = row0 + ty + 16 * a;
                if (row >= N) continue;
                const float hn = xh[row];
#pragma unroll
                for (int b = 0; b < 4; ++b) {
                    const int q = qg + tx + 16 * b;
                    if (q >= nq) continue;
                    const float s = acc[a][b] - hn;
                    if (s > thr[q]) {
                        const int pos = atomicAdd(&cnt[q], 1);
                        if (pos < kBufCap) mybuf[(size_t)q * kBufCap + pos] = pack_entry(s, (int32_t)row);
                    }
                }
            }
        }
        __syncthreads();
        for (int q = warp; q < nq; q += 8)
            if (cnt[q] > kBufCap - kTileRows)
                warp_compact<kBufCap>(mybuf + (size_t)q * kBufCap, &cnt[q], &thr[q], &thr_g[q], kp,
                                      top1 + (size_t)q * gridDim.x, blockIdx.x, gridDim.x, false);
        __syncthreads();
    }
    for (int q = warp; q < nq; q += 8)
        warp_compact<kBufCap>(mybuf + (size_t)q * kBufCap, &cnt[q], &thr[q], &thr_g[q], kp,
                              top1 + (size_t)q * gridDim.x, blockIdx.x, gridDim.x, true);
    __syncthreads();
    for (int q = tid; q < nq; q += blockDim.x) buf_cnt[(size_t)blockIdx.x * kScanQ + q] = cnt[q];
}

// ------------------------------------------------------------------------------------------
// Merge: per query, the k' best entries over all candidate lists of the pass.  A list holds up to
// `stride` entries as the scan left them; entries below the query's shared score bound (a lower
// bound of its global k'-th best) are dropped on the way in.  What is left is staged in shared
// memory when it fits; radix select on the 32-bit ordered score, then a collection pass.
// ------------------------------------------------------------------------------------------
constexpr int kMergeStage = 8192;                  // entries staged in shared memory
constexpr int kMergeStageMax = 24576;              // ... when few rows were scanned, so that every row may be an entry

struct MergeSrc {
    const u64 *buf;                                // lists of this query: list p at buf + p * list_stride
    const int32_t *cnt;                            // cnt[p * cnt_stride]
    size_t list_stride;
    int cnt_stride, n_lists, cap, total;
    uint32_t g0;                                   // entries whose ordered score is below it do not count
    const u64 *stage;                              // non-null: all entries are in stage[0 .. total)
    __device__ __forceinline__ int span() const { return stage ? total : n_lists * cap; }
    __device__ __forceinline__ bool get(int idx, u64 &ent) const {
        if (stage) { ent = stage[idx]; return true; }
        const int p = idx / cap, e = idx - p * cap;
        if (e >= cnt[(size_t)p * cnt_stride]) return false;
        ent = buf[(size_t)p * list_stride + e];
        return (uint32_t)(ent >> 32) >= g0;
    }
};

__global__ void __launch_bounds__(1024, 2)
merge_select_kernel(const int *__restrict__ n_active, int n_lists, int stride, int kp, int stage_cap,
                    const u64 *__restrict__ buf, const int32_t *__restrict__ buf_cnt, size_t buf_pass_stride,
                    size_t cnt_pass_stride, const uint32_t *__restrict__ thr_g, int32_t *cand_id, float *cand_score,
                    int32_t *cand_n, float *cand_sk) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    u64 *stage = reinterpret_cast<u64 *>(smem_raw);
    __shared__ unsigned hist[256];
    __shared__ uint32_t s_prefix, s_mask;
    __shared__ int s_remaining, s_total, s_gt, s_eq;
    const int m = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (m >= *n_active) return;
    const int pass = m / kScanQ, q = m - pass * kScanQ;    // every pass of the batch has its own lists
    buf += (size_t)pass * buf_pass_stride;
    buf_cnt += (size_t)pass * cnt_pass_stride;

    if (tid == 0) { s_total = 0; s_gt = 0; s_eq = 0; }
    __syncthreads();
    const uint32_t g0 = thr_g[m];
    // warp w takes the lists w, w + 32, ...: their counts come in with one load per 32 lists.  The
    // entries are few per list and scattered over many lists, so the staging is bound by load
    // latency: two lists at a time, up to 64 entries of each in flight per round (two blocks of 1024
    // threads share an SM, which leaves 32 registers a thread).
    for (int p0 = warp; p0 < n_lists; p0 += 32 * 32) {
        int my_c = 0;
        if (p0 + 32 * lane < n_lists) {
            my_c = buf_cnt[(size_t)(p0 + 32 * lane) * kScanQ + q];
            if (my_c > stride) my_c = stride;
        }
        for (int i = 0; i < 32 && p0 + 32 * i < n_lists; i += 2) {
            const int ca = __shfl_sync(0xffffffffu, my_c, i);
            const int cb = __shfl_sync(0xffffffffu, my_c, (i + 1) & 31);
            const bool two = i + 1 < 32 && p0 + 32 * (i + 1) < n_lists;
            const int c0 = ca, c1 = two ? cb : 0;
            const u64 *list0 = buf + ((size_t)(p0 + 32 * i) * kScanQ + q) * stride;
            const u64 *list1 = list0 + (size_t)32 * kScanQ * stride;          // list p + 32 (read only when two)
            const int cmax = c0 > c1 ? c0 : c1;
            for (int e0 = 0; e0 < cmax; e0 += 64) {
                u64 ent[4];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const int idx = e0 + 32 * u + lane;
                    ent[u] = idx < c0 ? list0[idx] : 0ull;
                    ent[2 + u] = idx < c1 ? list1[idx] : 0ull;
                }
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    if (e0 + 32 * (u & 1) >= (u < 2 ? c0 : c1)) continue;      // warp-uniform: nothing was loaded
                    const bool keep = ent[u] != 0ull && (uint32_t)(ent[u] >> 32) >= g0;
                    const unsigned mask = __ballot_sync(0xffffffffu, keep);
                    if (mask == 0u) continue;
                    int base = 0;
                    if (lane == 0) base = atomicAdd(&s_total, __popc(mask));
                    base = __shfl_sync(0xffffffffu, base, 0) + __popc(mask & ((1u << lane) - 1u));
                    if (keep && base < stage_cap) stage[base] = ent[u];
                }
            }
        }
    }
    __syncthreads();
    MergeSrc src;
    src.buf = buf + (size_t)q * stride;
    src.cnt = buf_cnt + q;
    src.list_stride = (size_t)kScanQ * stride;
    src.cnt_stride = kScanQ;
    src.n_lists = n_lists; src.cap = stride; src.g0 = g0; src.total = s_total;
    src.stage = (s_total <= stage_cap) ? stage : nullptr;
    const int total = src.total, span = src.span();

    uint32_t T = 0;                                // ordered score of the k'-th best (0: keep all)
    if (total >= kp) {
        if (tid == 0) { s_prefix = 0; s_mask = 0; s_remaining = kp; }
        for (int dg = 3; dg >= 0; --dg) {
            if (tid < 256) hist[tid] = 0;
            __syncthreads();
            const uint32_t prefix = s_prefix, mask = s_mask;
            for (int idx = tid; idx < span; idx += blockDim.x) {
                u64 ent;
                if (src.get(idx, ent)) {
                    const uint32_t o = (uint32_t)(ent >> 32);
                    if ((o & mask) == prefix) atomicAdd(&hist[(o >> (8 * dg)) & 255u], 1u);
                }
            }
            __syncthreads();
            if (warp == 0) {                       // walk the digits from the top: largest scores first
                int rem = s_remaining;
                const int b = radix_digit_walk(hist, rem, true);
                if (lane == 0) {
                    s_remaining = rem;
                    s_prefix = prefix | ((uint32_t)b << (8 * dg));
                    s_mask = mask | (0xffu << (8 * dg));
                }
            }
            __syncthreads();
        }
        T = s_prefix;
    }
    // entries above T all go in; entries equal to T fill what is left
    const int keep = total < kp ? total : kp;
    for (int idx = tid; idx < span; idx += blockDim.x) {
        u64 ent;
        if (src.get(idx, ent)) {
            const uint32_t o = (uint32_t)(ent >> 32);
            if (o > T || total < kp) {
                const int pos = atomicAdd(&s_gt, 1);
                cand_id[(size_t)m * kMaxKp + pos] = entry_row(ent);
                cand_score[(size_t)m * kMaxKp + pos] = o2f(o);
            }
        }
    }
    __syncthreads();
    const int n_gt = s_gt;
    if (total >= kp) {
        for (int idx = tid; idx < span; idx += blockDim.x) {
            u64 ent;
            if (src.get(idx, ent) && (uint32_t)(ent >> 32) == T) {
                const int pos = n_gt + atomicAdd(&s_eq, 1);
                if (pos < kp) {
                    cand_id[(size_t)m * kMaxKp + pos] = entry_row(ent);
                    cand_score[(size_t)m * kMaxKp + pos] = o2f(T);
                }
            }
        }
    }
    if (tid == 0) {
        cand_n[m] = keep;
        // fewer than k' entries: no row outside them scored above the bound the scan started from
        // (-inf for the corpus scan: every row is a candidate; the tolerance's bound for the probe)
        cand_sk[m] = (total >= kp) ? o2f(T) : o2f(g0);
    }
}

// ------------------------------------------------------------------------------------------
// Exact distances of a query's candidates and the final order.
// ------------------------------------------------------------------------------------------
__device__ __forceinline__ double exact_sqdist_warp(const float *__restrict__ q_sm,
                                                    const float *__restrict__ x, int d) {
    const int lane = threadIdx.x & 31;
    double acc = 0.0;
    for (int j = lane; j < d; j += 32) {
        const double df = (double)q_sm[j] - (double)x[j];
        acc = fma(df, df, acc);
    }
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
    return acc;
}

// The distance of the handle's metric in fp64: squared Euclidean, or -(q . x) for the inner product.
__device__ __forceinline__ double exact_dist_warp(const float *__restrict__ q_sm, const float *__restrict__ x, int d,
                                                  int ip) {
    if (!ip) return exact_sqdist_warp(q_sm, x, d);
    const int lane = threadIdx.x & 31;
    double acc = 0.0;
    for (int j = lane; j < d; j += 32) acc = fma((double)q_sm[j], (double)x[j], acc);
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
    return -acc;
}

constexpr int kRerankMax = kCollectCap;            // entries the sort buffers hold

// mode 0: candidates of the coarse scan (+ certificate); mode 1: rows collected by the exact pass
__global__ void __launch_bounds__(1024)
rerank_kernel(DevState *st, int mode, const float *__restrict__ corpus, const float *__restrict__ queries,
              int d, int k, long long N, const int32_t *__restrict__ miss_list,
              const int32_t *__restrict__ cand_id, const int32_t *__restrict__ cand_n,
              const float *__restrict__ cand_sk, const float *__restrict__ qbn,
              const float *__restrict__ qerr, int32_t *res_ids, double *res_dists, int32_t *fail_list,
              float *fail_radius, const int32_t *__restrict__ coll_id, const int32_t *__restrict__ coll_n, int ip,
              int32_t *over_list) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *sd = reinterpret_cast<double *>(smem_raw);                 // kRerankMax
    int *sid = reinterpret_cast<int *>(sd + kRerankMax);               // kRerankMax
    float *q_sm = reinterpret_cast<float *>(sid + kRerankMax);         // d
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

    int m, n;
    const int32_t *ids;
    if (mode == 0) {
        m = blockIdx.x;
        if (m >= st->n_miss) return;
        n = cand_n[m];
        ids = cand_id + (size_t)m * kMaxKp;
    } else {
        const int f = blockIdx.x;
        if (f >= st->n_fail) return;
        m = fail_list[f];
        n = coll_n[f];
        if (n > kCollectCap) {                     // more rows inside the radius than the collection holds:
            if (tid == 0) over_list[atomicAdd(&st->n_over, 1)] = f;      // answered by the streaming pass below
            return;
        }
        if (tid == 0) atomicAdd((u64 *)&st->fallback_rows, (u64)n);
        ids = coll_id + (size_t)f * kCollectCap;
    }
    const float *q = queries + (size_t)miss_list[m] * d;
    for (int j = tid; j < d; j += blockDim.x) q_sm[j] = q[j];
    int n2 = 1;
    while (n2 < n) n2 <<= 1;
    for (int e = tid; e < n2; e += blockDim.x) { sd[e] = INFINITY; sid[e] = 0x7fffffff; }
    __syncthreads();
    // one candidate row per warp at a time: the gathers are bound by latency, so the block is wide
    for (int c = warp; c < n; c += (int)(blockDim.x >> 5)) {
        const int row = ids[c];
        const double v = exact_dist_warp(q_sm, corpus + (size_t)row * d, d, ip);
        if (lane == 0) { sd[c] = v; sid[c] = row; }
    }
    block_sort_asc(sd, sid, n2);
    if (n < k) {                                    // cannot happen: k <= N and the sets hold >= k rows
        if (tid == 0) atomicCAS(&st->error, 0, PROX_ERR_INTERNAL);
        return;
    }
    for (int r = tid; r < k; r += blockDim.x) {
        res_ids[(size_t)m * k + r] = sid[r];
        res_dists[(size_t)m * k + r] = sd[r];
    }
    if (mode == 0 && tid == 0) {
        const float sk = cand_sk[m];
        bool certified = true;
        if ((long long)n < N) {                     // rows outside the candidate set exist
            // coarse distance of any outside row >= |bf16 q|^2 - 2 sk, less the fp32 slack of the
            // accumulated dot product and of the stored norms
            const double qn = sqrt((double)qbn[m]), xn = (double)st->xn_max;
            const double slack = 4.0 * (double)(d + 16) * 5.9604644775390625e-08 *
                                 (2.0 * qn * xn + xn * xn + qn * qn);
            if (ip) {
                // inner product: q.x = bf16(q).bf16(x) + (q - bf16 q).x + bf16(q).(x - bf16 x), and no
                // outside row has a coarse product above sk: q.x <= sk + a |x| + |bf16 q| e + slack
                const double a = (double)qerr[m], e = (double)st->e_max;
                const double upper = (double)sk + a * (xn + e) + qn * e + slack;
                certified = sd[k - 1] < -upper;
            } else {
                const double cprime = (double)qbn[m] - 2.0 * (double)sk - slack;
                const double g = (double)qerr[m] + (double)st->e_max;
                const double root = cprime > 0.0 ? sqrt(cprime) : 0.0;
                const double lower = root > g ? (root - g) * (root - g) : 0.0;
                certified = sd[k - 1] < lower;
            }
        }
        if (!certified) {
            const int f = atomicAdd(&st->n_fail, 1);
            fail_list[f] = m;
            const float rk = (float)sd[k - 1];
            fail_radius[f] = rk + fabsf(rk) * 1e-6f + 1e-30f;             // rounded up (the value may be negative)
            atomicAdd((u64 *)&st->uncertified, 1ull);
        }
    }
}

// ------------------------------------------------------------------------------------------
// Re-ranking of a hit (Section 3.3, re-ranking factor rho > 1): the k stored rows of the matched
// key measured against the current query in fp64, sorted by (distance, row id), the k_out
// nearest returned.  kind 1: key stored before the batch (list in the value slots); kind 2: key
// inserted earlier in this batch (list in the batch's results).  Stored id -1 (a pre-loaded key
// without a list) sorts last and comes back as -1 with an infinite distance.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
hit_rerank_kernel(int B, int d, int k, int k_out, int kind, const float *__restrict__ corpus,
                  const float *__restrict__ queries, const int32_t *__restrict__ src,
                  const int32_t *__restrict__ src_kind, const int32_t *__restrict__ miss_rank,
                  const int32_t *__restrict__ val_ids, const int32_t *__restrict__ res_ids, int64_t *out_ids,
                  float *out_dists, int ip) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *sd = reinterpret_cast<double *>(smem_raw);                 // kMaxFetch
    int *sid = reinterpret_cast<int *>(sd + kMaxFetch);                // kMaxFetch
    float *q_sm = reinterpret_cast<float *>(sid + kMaxFetch);          // d
    const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (i >= B || src_kind[i] != kind) return;
    const int32_t *ids = kind == 1 ? val_ids + (size_t)src[i] * k : res_ids + (size_t)miss_rank[src[i]] * k;
    for (int j = tid; j < d; j += blockDim.x) q_sm[j] = queries[(size_t)i * d + j];
    int n2 = 1;
    while (n2 < k) n2 <<= 1;
    for (int e = tid; e < n2; e += blockDim.x) { sd[e] = INFINITY; sid[e] = 0x7fffffff; }
    __syncthreads();
    for (int c = warp; c < k; c += 8) {
        const int row = ids[c];
        if (row < 0) continue;
        const double v = exact_dist_warp(q_sm, corpus + (size_t)row * d, d, ip);
        if (lane == 0) { sd[c] = v; sid[c] = row; }
    }
    block_sort_asc(sd, sid, n2);
    for (int r = tid; r < k_out; r += blockDim.x) {
        const bool have = sid[r] != 0x7fffffff;
        out_ids[(size_t)i * k_out + r] = have ? (int64_t)sid[r] : -1;
        out_dists[(size_t)i * k_out + r] = have ? (float)sd[r] : INFINITY;
    }
}

// ------------------------------------------------------------------------------------------
// Exact pass for uncertified queries: every corpus row within the radius (the exact k-th
// candidate distance) in fp32 difference form (inner product: fp32 sum of products, negated),
// with the fp32 rounding margin on top.  Eight queries per sweep of the corpus; one warp per row.
// `limit` holds, per query of the group, the largest fp32 value that is still collected (radius
// and margins folded in by the caller; -inf for an empty place in the group).
// ------------------------------------------------------------------------------------------
constexpr int kFallbackGroup = 8;

// Rows warp, warp + nwarps, ... of the corpus against NG queries held in shared memory (NG is the
// number of queries actually in the group, rounded up to 1, 2, 4 or 8, so that a lone failing
// query costs one query's arithmetic and the pass stays bound by the corpus read).
template <int NG, bool IP>
__device__ __forceinline__ void fallback_rows(const float *__restrict__ corpus, long long N, int d, long long warp,
                                              long long nwarps, const float *q_sm, const float *limit,
                                              int32_t *coll_id, int32_t *coll_n, int g0) {
    const int lane = threadIdx.x & 31;
    for (long long r = warp; r < N; r += nwarps) {
        const float4 *x = reinterpret_cast<const float4 *>(corpus + (size_t)r * d);
        float acc[NG];
#pragma unroll
        for (int f = 0; f < NG; ++f) acc[f] = 0.f;
        for (int j = lane; j < d / 4; j += 32) {
            const float4 xv = __ldcs(&x[j]);                       // streamed once: do not keep it in cache
#pragma unroll
            for (int f = 0; f < NG; ++f) {
                const float4 qv = *reinterpret_cast<const float4 *>(&q_sm[f * d + 4 * j]);
                if constexpr (IP) {
                    acc[f] = fmaf(-qv.x, xv.x, fmaf(-qv.y, xv.y, fmaf(-qv.z, xv.z, fmaf(-qv.w, xv.w, acc[f]))));
                } else {
                    const float d0 = qv.x - xv.x, d1 = qv.y - xv.y, d2 = qv.z - xv.z, d3 = qv.w - xv.w;
                    acc[f] = fmaf(d0, d0, fmaf(d1, d1, fmaf(d2, d2, fmaf(d3, d3, acc[f]))));
                }
            }
        }
#pragma unroll
        for (int f = 0; f < NG; ++f)
#pragma unroll
            for (int s = 16; s > 0; s >>= 1) acc[f] += __shfl_xor_sync(0xffffffffu, acc[f], s);
        if (lane < NG) {
            float mine = 0.f;
#pragma unroll
            for (int f = 0; f < NG; ++f)
                if (f == lane) mine = acc[f];
            if (mine <= limit[lane]) {
                const int pos = atomicAdd(&coll_n[g0 + lane], 1);
                if (pos < kCollectCap) coll_id[(size_t)(g0 + lane) * kCollectCap + pos] = (int32_t)r;
            }
        }
    }
}

// The same sweep over the bf16 copy of the corpus (half the bytes): |sqrt(coarse) - sqrt(exact)| is
// at most the rounding error of the row, so the caller passes radii widened by that error and
// every row within the exact radius is still collected (a few more with it).
template <int NG, bool IP>
__device__ __forceinline__ void fallback_rows_bf16(const __nv_bfloat16 *__restrict__ xb, long long N, int d,
                                                   long long warp, long long nwarps, const float *q_sm,
                                                   const float *limit, int32_t *coll_id,
                                                   int32_t *coll_n, int g0) {
    constexpr int U = NG <= 2 ? 4 : 2;                 // rows in flight per warp: the sweep is bound by load latency
    const int lane = threadIdx.x & 31;
    for (long long r0 = warp; r0 < N; r0 += (long long)U * nwarps) {
        float acc[U][NG];
#pragma unroll
        for (int u = 0; u < U; ++u)
#pragma unroll
            for (int f = 0; f < NG; ++f) acc[u][f] = 0.f;
        for (int j = lane; j < d / 8; j += 32) {
            uint4 w[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long r = r0 + (long long)u * nwarps;
                w[u] = r < N ? __ldcs(reinterpret_cast<const uint4 *>(xb + (size_t)r * d) + j) : make_uint4(0u, 0u, 0u, 0u);
            }
#pragma unroll
            for (int f = 0; f < NG; ++f) {
                const float4 qa = *reinterpret_cast<const float4 *>(&q_sm[f * d + 8 * j]);
                const float4 qb2 = *reinterpret_cast<const float4 *>(&q_sm[f * d + 8 * j + 4]);
#pragma unroll
                for (int u = 0; u < U; ++u) {
                    const uint32_t ww[4] = {w[u].x, w[u].y, w[u].z, w[u].w};   // eight bf16
                    const float x0 = __uint_as_float(ww[0] << 16), x1 = __uint_as_float(ww[0] & 0xffff0000u);
                    const float x2 = __uint_as_float(ww[1] << 16), x3 = __uint_as_float(ww[1] & 0xffff0000u);
                    const float x4 = __uint_as_float(ww[2] << 16), x5 = __uint_as_float(ww[2] & 0xffff0000u);
                    const float x6 = __uint_as_float(ww[3] << 16), x7 = __uint_as_float(ww[3] & 0xffff0000u);
                    if constexpr (IP) {
                        const float a = fmaf(-qa.x, x0, fmaf(-qa.y, x1, fmaf(-qa.z, x2, fmaf(-qa.w, x3, acc[u][f]))));
                        acc[u][f] = fmaf(-qb2.x, x4, fmaf(-qb2.y, x5, fmaf(-qb2.z, x6, fmaf(-qb2.w, x7, a))));
                    } else {
                        const float d0 = qa.x - x0, d1 = qa.y - x1, d2 = qa.z - x2, d3 = qa.w - x3;
                        const float d4 = qb2.x - x4, d5 = qb2.y - x5, d6 = qb2.z - x6, d7 = qb2.w - x7;
                        const float a = fmaf(d0, d0, fmaf(d1, d1, fmaf(d2, d2, fmaf(d3, d3, acc[u][f]))));
                        acc[u][f] = fmaf(d4, d4, fmaf(d5, d5, fmaf(d6, d6, fmaf(d7, d7, a))));
                    }
                }
            }
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const long long r = r0 + (long long)u * nwarps;
#pragma unroll
            for (int f = 0; f < NG; ++f)
#pragma unroll
                for (int s = 16; s > 0; s >>= 1) acc[u][f] += __shfl_xor_sync(0xffffffffu, acc[u][f], s);
            if (lane < NG && r < N) {
                float mine = 0.f;
#pragma unroll
                for (int f = 0; f < NG; ++f)
                    if (f == lane) mine = acc[u][f];
                if (mine <= limit[lane]) {
                    const int pos = atomicAdd(&coll_n[g0 + lane], 1);
                    if (pos < kCollectCap) coll_id[(size_t)(g0 + lane) * kCollectCap + pos] = (int32_t)r;
                }
            }
        }
    }
}

// Between the two sweeps of the exact pass: a query whose widened radius over the bf16 copy took
// in more rows than the collection holds is swept again over the fp32 rows with the exact radius.
__global__ void __launch_bounds__(1024)
fallback_mark_kernel(const DevState *st, int32_t *coll_n, int32_t *redo) {
    __shared__ int any;
    const int f = threadIdx.x;
    if (f == 0) any = 0;
    __syncthreads();
    const bool over = f < st->n_fail && coll_n[f] > kCollectCap;
    redo[f] = over ? 1 : 0;
    if (over) { coll_n[f] = 0; any = 1; }
    __syncthreads();
    if (f == 0) redo[kMaxBatch] = any;
}

template <int NG, bool IP>
__device__ __forceinline__ void fallback_sweep(const float *__restrict__ corpus, const __nv_bfloat16 *__restrict__ xb,
                                               long long N, int d, long long warp, long long nwarps, const float *q_sm,
                                               const float *limit, int32_t *coll_id, int32_t *coll_n, int g0) {
    if (xb != nullptr) fallback_rows_bf16<NG, IP>(xb, N, d, warp, nwarps, q_sm, limit, coll_id, coll_n, g0);
    else fallback_rows<NG, IP>(corpus, N, d, warp, nwarps, q_sm, limit, coll_id, coll_n, g0);
}

template <bool IP>
__global__ void __launch_bounds__(256)
fallback_collect_kernel(DevState *st, const float *__restrict__ corpus, const __nv_bfloat16 *__restrict__ xb,
                        const int32_t *__restrict__ redo,
                        const float *__restrict__ queries, long long N, int d, const int32_t *__restrict__ miss_list,
                        const int32_t *__restrict__ fail_list, const float *__restrict__ fail_radius,
                        const float *__restrict__ qbn, const float *__restrict__ qerr,
                        int32_t *coll_id, int32_t *coll_n) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *q_sm = reinterpret_cast<float *>(smem_raw);                  // kFallbackGroup x d
    __shared__ float limit[kFallbackGroup];
    const int n_fail = st->n_fail;
    if (n_fail == 0) return;
    if (redo != nullptr && redo[kMaxBatch] == 0) return;                // second sweep: nothing overflowed
    const int tid = threadIdx.x;
    const long long warp = ((long long)blockIdx.x * blockDim.x + tid) >> 5;
    const long long nwarps = ((long long)gridDim.x * blockDim.x) >> 5;
    const float margin = (float)(d + 8) * 1.1920929e-07f;              // (d + 8) * 2^-23, relative

    for (int g0 = 0; g0 < n_fail; g0 += kFallbackGroup) {
        const int ng = (n_fail - g0 < kFallbackGroup) ? n_fail - g0 : kFallbackGroup;
        __syncthreads();
        for (int idx = tid; idx < kFallbackGroup * d; idx += blockDim.x) {
            const int f = idx / d, j = idx - f * d;
            q_sm[idx] = (f < ng) ? queries[(size_t)miss_list[fail_list[g0 + f]] * d + j] : 0.f;
        }
        if (tid < kFallbackGroup) {
            bool live = tid < ng;
            if (redo != nullptr && live && redo[g0 + tid] == 0) live = false;   // settled by the first sweep
            float lim = -INFINITY;
            if (live) {
                const float rad = fail_radius[g0 + tid];
                if constexpr (IP) {
                    // |q| (|x| + e) bounds the sum of |q_j x_j|: margin times it covers the fp32 sum; over the
                    // bf16 copy the row's rounding error moves the product by at most |q| e_max more
                    const int m = fail_list[g0 + tid];
                    const float qn = (sqrtf(qbn[m]) + qerr[m]) * (1.f + 2e-7f);
                    const float xn = (st->xn_max + st->e_max) * (1.f + 2e-7f);
                    lim = rad + margin * qn * xn * (1.f + 2e-7f) + 1e-30f;
                    if (xb != nullptr) lim += qn * st->e_max * (1.f + 4e-7f);
                } else if (xb != nullptr) {                        // widened by the rows' rounding error, rounded up
                    const float w = sqrtf(rad) * (1.f + 2e-7f) + st->e_max * (1.f + 2e-7f);
                    lim = w * w * (1.f + 2e-7f) * (1.f + margin) + 1e-30f;
                } else {
                    lim = rad * (1.f + margin) + 1e-30f;
                }
            }
            limit[tid] = lim;
        }
        __syncthreads();
        if (ng == 1) fallback_sweep<1, IP>(corpus, xb, N, d, warp, nwarps, q_sm, limit, coll_id, coll_n, g0);
        else if (ng == 2) fallback_sweep<2, IP>(corpus, xb, N, d, warp, nwarps, q_sm, limit, coll_id, coll_n, g0);
        else if (ng <= 4) fallback_sweep<4, IP>(corpus, xb, N, d, warp, nwarps, q_sm, limit, coll_id, coll_n, g0);
        else fallback_sweep<8, IP>(corpus, xb, N, d, warp, nwarps, q_sm, limit, coll_id, coll_n, g0);
    }
}

// ------------------------------------------------------------------------------------------
// Last resort of the exact pass: a query with more rows inside its radius than the collection
// holds (thousands of copies of one row next to the query, say).  Every block walks its own
// contiguous share of the corpus, measures every row exactly (fp64) and keeps the rows that are
// still among its k nearest by (distance, row id) in a shared-memory buffer that is sorted and
// cut to k whenever it fills up; the block that delivers its list last merges all lists the same
// way and writes the answer.  No row is ever dropped unseen, so the result is exact whatever the
// number of ties.  Queries are taken one after the other (up to kOverMax per batch); the pass
// costs one reading of the fp32 corpus per query and runs for pathological inputs only.
// ------------------------------------------------------------------------------------------
constexpr int kOverBuf = 4096;

// Sorts the n entries of the buffer by (distance, row) and keeps the first k; returns how many stay.
__device__ int over_compact(double *bd, int *bid, int n, int k) {
    int n2 = 2;
    while (n2 < n) n2 <<= 1;                   // (n <= kOverBuf, a power of two)
    for (int e = n + threadIdx.x; e < n2; e += blockDim.x) { bd[e] = INFINITY; bid[e] = 0x7fffffff; }
    block_sort_asc(bd, bid, n2);
    return n < k ? n : k;
}

template <bool IP>
__global__ void __launch_bounds__(1024)
overflow_topk_kernel(DevState *st, const float *__restrict__ corpus, const float *__restrict__ queries, long long N,
                     int d, int k, const int32_t *__restrict__ miss_list, const int32_t *__restrict__ fail_list,
                     const float *__restrict__ fail_radius, const int32_t *__restrict__ over_list, double *over_d,
                     int32_t *over_id, unsigned *over_ticket, int32_t *res_ids, double *res_dists, int direct) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    double *bd = reinterpret_cast<double *>(smem_raw);                 // kOverBuf
    int *bid = reinterpret_cast<int *>(bd + kOverBuf);                 // kOverBuf
    float *q_sm = reinterpret_cast<float *>(bid + kOverBuf);           // d
    __shared__ int s_cnt;
    __shared__ unsigned s_last;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
    // direct: the whole database call of a small batch over a small corpus (every miss, no radius)
    int n_over = direct ? st->n_miss : st->n_over;
    if (n_over == 0) return;
    if (direct && blockIdx.x == 0 && tid == 0) st->scan_batches++;
    if (n_over > kOverMax) {                   // beyond what the lists hold: those queries stay unanswered, and say so
        if (blockIdx.x == 0 && tid == 0) {
            atomicAdd((u64 *)&st->unresolved, (u64)(n_over - kOverMax));
            atomicCAS(&st->error, 0, PROX_ERR_INTERNAL);
        }
        n_over = kOverMax;
    }
    const long long per = (N + gridDim.x - 1) / gridDim.x;
    const long long r0 = (long long)blockIdx.x * per, r1 = r0 + per < N ? r0 + per : N;

    for (int o = 0; o < n_over; ++o) {
        const int f = direct ? o : over_list[o], m = direct ? o : fail_list[f];
        __syncthreads();
        for (int j = tid; j < d; j += blockDim.x) q_sm[j] = queries[(size_t)miss_list[m] * d + j];
        if (tid == 0) s_cnt = 0;
        // a row counts while (distance, row) <= (bound_d, bound_id): first the radius, then the block's k-th nearest
        double bound_d = direct ? INFINITY : (double)fail_radius[f];
        int bound_id = 0x7fffffff;
        __syncthreads();
        for (long long base = r0; base < r1; base += nwarps) {
            const long long row = base + warp;
            if (row < r1) {
                const double v = exact_dist_warp(q_sm, corpus + (size_t)row * d, d, IP ? 1 : 0);
                if (lane == 0 && (v < bound_d || (v == bound_d && (int)row <= bound_id))) {
                    const int pos = atomicAdd(&s_cnt, 1);
                    bd[pos] = v;
                    bid[pos] = (int)row;
                }
            }
            __syncthreads();
            const int n = s_cnt;
            if (n > kOverBuf - nwarps) {       // the next round could overflow: sort, keep k, tighten the bound
                const int keep = over_compact(bd, bid, n, k);
                if (keep == k) { bound_d = bd[k - 1]; bound_id = bid[k - 1]; }
                __syncthreads();
                if (tid == 0) s_cnt = keep;
                __syncthreads();
            }
        }
        const int mine = over_compact(bd, bid, s_cnt, k);
        double *my_d = over_d + ((size_t)o * gridDim.x + blockIdx.x) * k;
        int32_t *my_id = over_id + ((size_t)o * gridDim.x + blockIdx.x) * k;
        for (int e = tid; e < k; e += blockDim.x) {
            my_d[e] = e < mine ? bd[e] : INFINITY;
            my_id[e] = e < mine ? bid[e] : -1;
        }
        __threadfence();
        __syncthreads();
        if (tid == 0) s_last = (atomicAdd(&over_ticket[o], 1u) == gridDim.x - 1) ? 1u : 0u;
        __syncthreads();
        if (s_last) {                          // every block's list is in memory: merge them the same way
            __threadfence();
            int n = 0;
            const int total = (int)gridDim.x * k;
            for (int e0 = 0; e0 < total; e0 += kOverBuf - k) {
                const int chunk = total - e0 < kOverBuf - k ? total - e0 : kOverBuf - k;
                for (int e = tid; e < chunk; e += blockDim.x) {
                    bd[n + e] = __ldcg(over_d + (size_t)o * total + e0 + e);
                    const int id = __ldcg(over_id + (size_t)o * total + e0 + e);
                    bid[n + e] = id < 0 ? 0x7fffffff : id;
                }
                __syncthreads();
                n = over_compact(bd, bid, n + chunk, k);
                __syncthreads();
            }
            if (n < k || bid[k - 1] == 0x7fffffff) {     // cannot happen: at least k rows lie inside the radius
                if (tid == 0) atomicCAS(&st->error, 0, PROX_ERR_INTERNAL);
            } else {
                for (int r = tid; r < k; r += blockDim.x) {
                    res_ids[(size_t)m * k + r] = bid[r];
                    res_dists[(size_t)m * k + r] = bd[r];
                }
            }
            if (tid == 0) {
                over_ticket[o] = 0u;           // ready for the next batch
                if (!direct) atomicAdd((u64 *)&st->fallback_rows, (u64)N);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------
// Coarse tensor-core probe (the key distances of Algorithm 1, for large caches): the scan kernel run over
// the bf16 copies of the keys gives, per query, the kProbeKp slots with the best coarse scores;
// here their exact fp64 distances give the nearest safe slot, with the same kind of
// certificate as the corpus scan.  At-risk slots are left out (the fp64 probe measures them as
// full rows).  Only a safe minimum within tau matters to the resolve, so a query is settled if
//   - every valid slot was a candidate, or
//   - the best safe candidate is nearer than any slot outside the candidates can be, or
//   - no slot outside the candidates can be within tau.
// Otherwise the query is handed to the exact fp64 probe over all slots.
// ------------------------------------------------------------------------------------------
// Largest coarse squared distance that a pair whose true squared distance is at most tau can show:
// rounding to bf16 moves either vector by at most a resp. e, the fp32 sum and norms by the slack.
__device__ __forceinline__ double coarse_bound(double tau, double a, double e, double qn, double kn, int d) {
    const double slack = 4.0 * (double)(d + 16) * 5.9604644775390625e-08 * (2.0 * qn * kn + kn * kn + qn * qn);
    const double r = sqrt(tau) + a + e;
    return r * r * (1.0 + 1e-6) + slack * (1.0 + 1e-6) + 4e-7 * (qn * qn + kn * kn) + 1e-30;
}

__global__ void __launch_bounds__(128)
prep_probe_kernel(DevState *st, const float *__restrict__ queries, int B, int d, double tau, __nv_bfloat16 *pqb,
                  float *pqbn, float *pqerr, uint32_t *thr_g, uint32_t *top1, int n_blocks, int32_t *use_partial,
                  int32_t *n_cand) {
    __shared__ float red[2][4];
    const int m = blockIdx.x, tid = threadIdx.x;
    if (m == 0 && tid == 0) { st->n_probe = B; st->n_pfail = 0; st->n_pairs = 0; st->side_overflow = 0; }
    for (int i = tid; i < n_blocks; i += blockDim.x) top1[(size_t)m * n_blocks + i] = 0u;
    if (m >= B) {
        if (tid == 0) thr_g[m] = f2o(-INFINITY);
        for (int j = tid; j < d; j += blockDim.x) pqb[(size_t)m * d + j] = __float2bfloat16_rn(0.f);
        return;
    }
    if (tid == 0) { use_partial[m] = 0; n_cand[m] = 0; }
    const float *src = queries + (size_t)m * d;
    float nn = 0.f, ee = 0.f;
    for (int j = tid; j < d; j += blockDim.x) {
        const float v = src[j];
        const __nv_bfloat16 b = __float2bfloat16_rn(v);
        const float f = __bfloat162float(b);
        pqb[(size_t)m * d + j] = b;
        nn += f * f;
        ee += (v - f) * (v - f);
    }
#pragma unroll
    for (int s = 16; s > 0; s >>= 1) {
        nn += __shfl_xor_sync(0xffffffffu, nn, s);
        ee += __shfl_xor_sync(0xffffffffu, ee, s);
    }
    if ((tid & 31) == 0) { red[0][tid >> 5] = nn; red[1][tid >> 5] = ee; }
    __syncthreads();
    if (tid == 0) {
        const float n2 = red[0][0] + red[0][1] + red[0][2] + red[0][3];
        const float err = sqrtf(red[1][0] + red[1][1] + red[1][2] + red[1][3]) * 1.0001f;
        pqbn[m] = n2;
        pqerr[m] = err;
        // The scan starts from the tolerance's bound instead of an open threshold: a key whose coarse
        // score is below it cannot lie within tau, and only a key within tau matters to the lookup.
        // score = (|bf16 q|^2 - coarse distance) / 2, rounded down.
        const double T = coarse_bound(tau, (double)err, (double)st->ke_max, sqrt((double)n2), (double)st->kn_max, d);
        thr_g[m] = f2o(__double2float_rd(0.5 * ((double)n2 - T)));
    }
}

__global__ void __launch_bounds__(128)
probe_exact_kernel(DevState *st, const float *__restrict__ keys, const float *__restrict__ queries, int B, int d,
                   double tau, const int32_t *__restrict__ risk_pos, const int32_t *__restrict__ cand_id,
                   const float *__restrict__ cand_score, const int32_t *__restrict__ cand_n,
                   const float *__restrict__ cand_sk, const float *__restrict__ pqbn, const float *__restrict__ pqerr,
                   double *safe_min, int32_t *safe_arg, int32_t *use_partial, int32_t *pfail_list) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    float *q_sm = reinterpret_cast<float *>(smem_raw);
    __shared__ double w_d[4];
    __shared__ int w_s[4];
    __shared__ float w_f[4];
    __shared__ int w_i[4];
    __shared__ int s_list[kProbeKp], s_n;
    const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (i >= B) return;
    for (int j = tid; j < d; j += blockDim.x) q_sm[j] = queries[(size_t)i * d + j];
    if (tid == 0) s_n = 0;
    const int n = cand_n[i];                                  // <= kProbeKp <= blockDim.x
    // the safe candidate with the best coarse score first: its exact distance bounds the coarse
    // score of anything that could be nearer, and few of the other candidates reach that bound
    int my_slot = -1;
    float my_score = -INFINITY;
    if (tid < n) {
        const int slot = cand_id[(size_t)i * kMaxKp + tid];
        if (risk_pos[slot] < 0) { my_slot = slot; my_score = cand_score[(size_t)i * kMaxKp + tid]; }   // at-risk: measured elsewhere
    }
    float bf = my_score;
    int bi = my_slot >= 0 ? tid : 0x7fffffff;
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) {
        const float of = __shfl_xor_sync(0xffffffffu, bf, m);
        const int oi = __shfl_xor_sync(0xffffffffu, bi, m);
        if (of > bf || (of == bf && oi < bi)) { bf = of; bi = oi; }
    }
    if (lane == 0) { w_f[warp] = bf; w_i[warp] = bi; }
    __syncthreads();
    for (int w = 0; w < 4; ++w)
        if (w_f[w] > bf || (w_f[w] == bf && w_i[w] < bi)) { bf = w_f[w]; bi = w_i[w]; }
    double bd = INFINITY;
    int bs = 0x7fffffff;
    if (bi != 0x7fffffff) {                                   // (block-uniform)
        const int first = cand_id[(size_t)i * kMaxKp + bi];
        const double d1 = exact_sqdist_warp(q_sm, keys + (size_t)first * d, d);    // every warp computes it: no hand-over
        bd = d1;
        bs = first;
        const double qn2 = (double)pqbn[i];
        const double T = coarse_bound(d1, (double)pqerr[i], (double)st->ke_max, sqrt(qn2), (double)st->kn_max, d);
        const float s_min = __double2float_rd(0.5 * (qn2 - T));
        if (my_slot >= 0 && tid != bi && my_score >= s_min) s_list[atomicAdd(&s_n, 1)] = my_slot;
        __syncthreads();
        const int m = s_n;
        for (int c = warp; c < m; c += 4) {
            const int slot = s_list[c];
            const double v = exact_sqdist_warp(q_sm, keys + (size_t)slot * d, d);
            if (v < bd || (v == bd && slot < bs)) { bd = v; bs = slot; }
        }
    }
    __syncthreads();
    if (lane == 0) { w_d[warp] = bd; w_s[warp] = bs; }
    __syncthreads();
    if (tid == 0) {
        for (int w = 1; w < 4; ++w)
            if (w_d[w] < bd || (w_d[w] == bd && w_s[w] < bs)) { bd = w_d[w]; bs = w_s[w]; }
        const float sk = cand_sk[i];
        bool settled = true;
        if (sk != -INFINITY) {                                    // slots outside the candidate set exist
            const double qn = sqrt((double)pqbn[i]), kn = (double)st->kn_max;
            const double slack = 4.0 * (double)(d + 16) * 5.9604644775390625e-08 * (2.0 * qn * kn + kn * kn + qn * qn);
            const double cprime = (double)pqbn[i] - 2.0 * (double)sk - slack;
            const double g = (double)pqerr[i] + (double)st->ke_max;
            const double root = cprime > 0.0 ? sqrt(cprime) : 0.0;
            const double lower = root > g ? (root - g) * (root - g) : 0.0;    // no outside slot is nearer than this
            settled = (bd < lower) || (lower > tau);
        }
        safe_min[i] = bd;
        safe_arg[i] = (bs == 0x7fffffff) ? -1 : bs;
        if (!settled) {
            use_partial[i] = 1;
            pfail_list[atomicAdd(&st->n_pfail, 1)] = i;
            atomicAdd((u64 *)&st->probe_uncertified, 1ull);
        }
    }
}

// ------------------------------------------------------------------------------------------
// Launchers
// ------------------------------------------------------------------------------------------
void launch_convert_corpus(prox_handle *h, cudaStream_t s) {
    convert_corpus_kernel<<<h->num_sms * 8, 256, 0, s>>>(h->corpus, (long long)h->N, h->d, h->xb, h->xh,
                                                         h->st, metric_is_ip(h) ? 1 : 0);
    h->launches++;
}

void launch_prep_miss(prox_handle *h, const float *q, int B, cudaStream_t s) {
    int rows = ((B + kScanQ - 1) / kScanQ) * kScanQ;      // zero the padding rows of the last pass too
    if (rows > kMaxBatch) rows = kMaxBatch;
    prep_miss_kernel<<<rows, 128, 0, s>>>(h->st, q, B, h->d, h->miss_list, h->qb, h->qbn, h->qerr, h->thr_g,
                                          h->coll_n, h->top1, 4 * h->scan_ctas);
    h->launches++;
}

void launch_scan_pass(prox_handle *h, int pass, cudaStream_t s) {
    h->scan_lists = h->scan_ctas;                         // one candidate list per block and query
    h->scan_list_stride = kBufCap;
    scan_cc_kernel<<<h->scan_ctas, 256, 0, s>>>(h->st, h->xb, h->xh, h->qb, (long long)h->N, h->d, pass,
                                                h->kp, h->thr_g, h->top1, h->buf + (size_t)pass * h->buf_pass_stride,
                                                h->buf_cnt + (size_t)pass * h->cnt_pass_stride);
    h->launches++;
}

void launch_merge_select(prox_handle *h, int B, int for_probe, cudaStream_t s) {
    // a scan of few rows never tightens its bounds, so every row may still be in the lists: stage them all
    const long long rows = for_probe ? (long long)h->C : (long long)h->N;
    const int stage_cap = rows <= kMergeStageMax ? (int)((rows + 1023) / 1024 * 1024) : kMergeStage;
    merge_select_kernel<<<B, 1024, (size_t)stage_cap * 8, s>>>(for_probe ? &h->st->n_probe : &h->st->n_miss,
                                                         h->scan_lists, h->scan_list_stride, for_probe ? kProbeKp : h->kp, stage_cap,
                                                         h->buf, h->buf_cnt, h->buf_pass_stride, h->cnt_pass_stride, h->thr_g,
                                                         h->cand_id, h->cand_score, h->cand_n, h->cand_sk);
    h->launches++;
}

static size_t rerank_smem(int d) { return (size_t)kRerankMax * 12 + (size_t)d * 4; }

// Kernel attributes belong to a device: set when a handle is created there, not once per process.
void set_scan_kernel_attributes() {
    cudaFuncSetAttribute(merge_select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMergeStageMax * 8);
    cudaFuncSetAttribute(rerank_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)rerank_smem(4096));
    cudaFuncSetAttribute(fallback_collect_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFallbackGroup * 4096 * 4);
    cudaFuncSetAttribute(fallback_collect_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kFallbackGroup * 4096 * 4);
    cudaFuncSetAttribute(overflow_topk_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kOverBuf * 12 + 4096 * 4);
    cudaFuncSetAttribute(overflow_topk_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kOverBuf * 12 + 4096 * 4);
}

void launch_rerank(prox_handle *h, const float *q, int B, cudaStream_t s) {
    rerank_kernel<<<B, 1024, rerank_smem(h->d), s>>>(h->st, 0, h->corpus, q, h->d, h->k, (long long)h->N,
                                                    h->miss_list, h->cand_id, h->cand_n, h->cand_sk, h->qbn,
                                                    h->qerr, h->res_ids, h->res_dists, h->fail_list,
                                                    h->fail_radius, h->coll_id, h->coll_n, metric_is_ip(h) ? 1 : 0, h->over_list);
    h->launches++;
}

void launch_hit_rerank(prox_handle *h, const float *q, int B, int kind, int64_t *out_ids, float *out_dists,
                       cudaStream_t s) {
    const size_t smem = (size_t)kMaxFetch * 12 + (size_t)h->d * 4;
    hit_rerank_kernel<<<B, 256, smem, s>>>(B, h->d, h->k, h->k_out, kind, h->corpus, q, h->src, h->src_kind,
                                           h->miss_rank, h->val_ids, h->res_ids, out_ids, out_dists,
                                           metric_is_ip(h) ? 1 : 0);
    h->launches++;
}

void launch_fallback(prox_handle *h, const float *q, int B, cudaStream_t s) {
    auto collect = metric_is_ip(h) ? fallback_collect_kernel<true> : fallback_collect_kernel<false>;
    collect<<<h->num_sms * 4, 256, (size_t)kFallbackGroup * h->d * 4, s>>>(
        h->st, h->corpus, h->xb, nullptr, q, (long long)h->N, h->d, h->miss_list, h->fail_list, h->fail_radius,
        h->qbn, h->qerr, h->coll_id, h->coll_n);
    // the bf16 sweep reads half the bytes; what it cannot hold is swept again in fp32
    fallback_mark_kernel<<<1, 1024, 0, s>>>(h->st, h->coll_n, h->redo);
    collect<<<h->num_sms * 4, 256, (size_t)kFallbackGroup * h->d * 4, s>>>(
        h->st, h->corpus, nullptr, h->redo, q, (long long)h->N, h->d, h->miss_list, h->fail_list, h->fail_radius,
        h->qbn, h->qerr, h->coll_id, h->coll_n);
    h->launches += 3;
    rerank_kernel<<<B, 1024, rerank_smem(h->d), s>>>(h->st, 1, h->corpus, q, h->d, h->k, (long long)h->N,
                                                    h->miss_list, h->cand_id, h->cand_n, h->cand_sk, h->qbn,
                                                    h->qerr, h->res_ids, h->res_dists, h->fail_list,
                                                    h->fail_radius, h->coll_id, h->coll_n, metric_is_ip(h) ? 1 : 0, h->over_list);
    h->launches++;
    // queries whose collection overflowed even in the fp32 sweep (returns at once when there is none)
    auto over = metric_is_ip(h) ? overflow_topk_kernel<true> : overflow_topk_kernel<false>;
    over<<<h->scan_ctas, 1024, (size_t)kOverBuf * 12 + (size_t)h->d * 4, s>>>(
        h->st, h->corpus, q, (long long)h->N, h->d, h->k, h->miss_list, h->fail_list, h->fail_radius, h->over_list,
        h->over_d, h->over_id, h->over_ticket, h->res_ids, h->res_dists, 0);
    h->launches++;
}

// The database call of a small batch over a small corpus in one launch: every row measured in fp64
// for every miss, the k nearest by (distance, row id).  Exact by construction; stands in for the
// coarse scan, its merge, the rerank and the exact pass, whose launches would cost more than the work.
bool small_corpus_fits(const prox_handle *h, int B) {
    return B <= 4 && (long long)h->N * h->d <= (1LL << 24) && h->N >= h->k;
}

void launch_small_exact(prox_handle *h, const float *q, cudaStream_t s) {
    auto kern = metric_is_ip(h) ? overflow_topk_kernel<true> : overflow_topk_kernel<false>;
    kern<<<h->scan_ctas, 1024, (size_t)kOverBuf * 12 + (size_t)h->d * 4, s>>>(
        h->st, h->corpus, q, (long long)h->N, h->d, h->k, h->miss_list, h->fail_list, h->fail_radius, h->over_list,
        h->over_d, h->over_id, h->over_ticket, h->res_ids, h->res_dists, 1);
    h->launches++;
}

}  // namespace prox

namespace prox {
void launch_prep_probe(prox_handle *h, const float *q, int B, cudaStream_t s) {
    int rows = ((B + kScanQ - 1) / kScanQ) * kScanQ;
    if (rows > kMaxBatch) rows = kMaxBatch;
    prep_probe_kernel<<<rows, 128, 0, s>>>(h->st, q, B, h->d, (double)h->tau, h->pqb, h->pqbn, h->pqerr, h->thr_g, h->top1,
                                           4 * h->scan_ctas, h->use_partial, h->n_cand);
    h->launches++;
}

void launch_probe_exact(prox_handle *h, const float *q, int B, cudaStream_t s) {
    probe_exact_kernel<<<B, 128, (size_t)h->d * 4, s>>>(h->st, h->keys, q, B, h->d, (double)h->tau, h->risk_pos,
                                                         h->cand_id, h->cand_score, h->cand_n, h->cand_sk, h->pqbn, h->pqerr,
                                                         h->safe_min, h->safe_arg, h->use_partial, h->pfail_list);
    h->launches++;
}
}  // namespace prox
