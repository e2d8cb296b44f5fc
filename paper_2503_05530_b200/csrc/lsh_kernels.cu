// PROXIMITY-LSH (Section 3.2 of the paper): random-hyperplane hash of every batch query, and the
// lookup of Algorithm 1 inside the one bucket that the hash names.  Buckets are independent
// flat caches of b entries with their own FIFO / LRU eviction (Section 3.3.2), so the batch is
// replayed in query order per bucket, all buckets of the batch side by side:
//   lsh_hash_kernel     bit l of the bucket number = (q . r_l >= 0), dot products in fp64;
//   lsh_group_kernel    batch queries sorted by (bucket, index); one run per bucket;
//   lsh_resolve_kernel  one block per run: for each query of the run in index order, fp64
//                       distances to the bucket's resident keys (a key inserted earlier in the
//                       batch is resident like any other), nearest key, test <= tau, LRU touch
//                       or insertion with eviction of the bucket's oldest stamp;
//   lsh_finish_kernel   miss list in index order, counters.
// The outputs are those of the flat cache's resolve step, so the database call of the misses,
// the re-ranking and the write-back that follow are shared with it.
#include <cmath>

#include "prox_internal.h"
#include "topk_device.cuh"

namespace prox {

namespace {

constexpr int kLshMaxBucket = 64;

// fp64 dot product / squared distance of two fp32 vectors by one warp (every lane gets the sum).
__device__ __forceinline__ double warp_sum(double acc) {
#pragma unroll
    for (int m = 16; m > 0; m >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, m);
    return acc;
}

__global__ void __launch_bounds__(256)
lsh_hash_kernel(int B, int d, int L, const float *__restrict__ queries, const float *__restrict__ planes,
                int32_t *code) {
    __shared__ unsigned bits;
    const int i = blockIdx.x, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (i >= B) return;
    if (threadIdx.x == 0) bits = 0u;
    __syncthreads();
    const float *q = queries + (size_t)i * d;
    for (int l = warp; l < L; l += 8) {
        const float *r = planes + (size_t)l * d;
        double acc = 0.0;
        for (int j = lane; j < d; j += 32) acc += (double)q[j] * (double)r[j];
        acc = warp_sum(acc);
        if (lane == 0 && acc >= 0.0) atomicOr(&bits, 1u << l);
    }
    __syncthreads();
    if (threadIdx.x == 0) code[i] = (int32_t)bits;
}

__global__ void __launch_bounds__(1024)
lsh_group_kernel(int B, const int32_t *__restrict__ code, int32_t *order, int32_t *seg, int32_t *work) {
    __shared__ u64 s_key[kMaxBatch];
    __shared__ int s_val[kMaxBatch];
    __shared__ int warp_tot[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    s_key[tid] = tid < B ? (u64)(uint32_t)code[tid] : ~0ull;
    s_val[tid] = tid < B ? tid : 0x7fffffff;
    int n2 = 1;
    while (n2 < B) n2 <<= 1;
    block_sort_asc(s_key, s_val, n2);
    // a run starts where the bucket changes
    const bool head = tid < B && (tid == 0 || s_key[tid] != s_key[tid - 1]);
    const unsigned m = __ballot_sync(0xffffffffu, head);
    if (lane == 0) warp_tot[warp] = __popc(m);
    __syncthreads();
    int base = 0;
    for (int w = 0; w < warp; ++w) base += warp_tot[w];
    if (head) seg[base + __popc(m & ((1u << lane) - 1u))] = tid;
    if (tid < B) order[tid] = s_val[tid];
    if (tid == 0) {
        int n = 0;
        for (int w = 0; w < 32; ++w) n += warp_tot[w];
        seg[n] = B;
        work[0] = n; work[1] = 0; work[2] = 0;
    }
}

__global__ void __launch_bounds__(256)
lsh_resolve_kernel(const DevState *st, int B, int d, int b, double tau, int policy,
                   const float *__restrict__ queries, const int32_t *__restrict__ code,
                   const int32_t *__restrict__ order, const int32_t *__restrict__ seg, int32_t *work, float *keys,
                   u64 *stamp, int32_t *bucket_count, uint8_t *out_hit, int32_t *src, int32_t *src_kind,
                   int32_t *ins_slot, int32_t *evt_slot, float *evt_dist) {
    __shared__ double s_dist[kLshMaxBucket];
    __shared__ u64 s_stamp[kLshMaxBucket];
    __shared__ int s_owner[kLshMaxBucket];       // batch query that wrote the slot in this batch, or -1
    __shared__ int s_cnt, s_slot, s_evict, s_intra;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if ((int)blockIdx.x >= work[0]) return;
    const int r0 = seg[blockIdx.x], r1 = seg[blockIdx.x + 1];
    const long long bucket = (long long)(uint32_t)code[order[r0]];
    const long long slot0 = bucket * b;
    const long long clock0 = st->clock;
    if (tid < b) { s_stamp[tid] = stamp[slot0 + tid]; s_owner[tid] = -1; }
    if (tid == 0) { s_cnt = bucket_count[bucket]; s_evict = 0; s_intra = 0; }
    __syncthreads();

    for (int r = r0; r < r1; ++r) {
        const int i = order[r];
        const float *q = queries + (size_t)i * d;
        const int cnt = s_cnt;
        // distances to the resident keys of the bucket (Algorithm 1), difference form in fp64
        for (int s = warp; s < cnt; s += 8) {
            const float *key = keys + (size_t)(slot0 + s) * d;
            double acc = 0.0;
            for (int j = lane; j < d; j += 32) {
                const double df = (double)q[j] - (double)key[j];
                acc += df * df;
            }
            acc = warp_sum(acc);
            if (lane == 0) s_dist[s] = acc;
        }
        __syncthreads();
        if (tid == 0) {
            double best = INFINITY;
            int bs = -1;
            for (int s = 0; s < cnt; ++s)
                if (s_dist[s] < best) { best = s_dist[s]; bs = s; }          // the lowest slot wins a tie
            const u64 t = (u64)(clock0 + i);                                  // one stamp per query
            if (bs >= 0 && best <= tau) {                                     // threshold test
                out_hit[i] = 1;
                if (policy == PROX_LRU) s_stamp[bs] = t;
                const int own = s_owner[bs];
                src_kind[i] = own >= 0 ? 2 : 1;
                src[i] = own >= 0 ? own : (int)(slot0 + bs);
                if (own >= 0) ++s_intra;
                evt_slot[i] = (int)(slot0 + bs);
                evt_dist[i] = (float)best;
                ins_slot[i] = -1;
                s_slot = -1;
            } else {                                                          // miss: evict if full, insert
                int s;
                if (cnt < b) {
                    s = cnt;
                    s_cnt = cnt + 1;
                } else {
                    s = 0;
                    for (int e = 1; e < b; ++e)
                        if (s_stamp[e] < s_stamp[s]) s = e;
                    if (s_owner[s] >= 0) ins_slot[s_owner[s]] = -1;           // gone before the batch ends
                    ++s_evict;
                }
                s_stamp[s] = t;
                s_owner[s] = i;
                out_hit[i] = 0;
                src_kind[i] = 0; src[i] = -1;
                evt_slot[i] = (int)(slot0 + s);
                evt_dist[i] = INFINITY;
                ins_slot[i] = (int)(slot0 + s);
                s_slot = s;
            }
        }
        __syncthreads();
        const int s = s_slot;
        if (s >= 0) {                                                         // the query becomes the slot's key at once
            float *key = keys + (size_t)(slot0 + s) * d;
            for (int j = tid; j < d; j += blockDim.x) key[j] = q[j];
        }
        __syncthreads();
    }
    if (tid < b) stamp[slot0 + tid] = s_stamp[tid];
    if (tid == 0) {
        bucket_count[bucket] = s_cnt;
        if (s_evict) atomicAdd(&work[1], s_evict);
        if (s_intra) atomicAdd(&work[2], s_intra);
    }
}

__global__ void __launch_bounds__(1024)
lsh_finish_kernel(DevState *st, int B, const uint8_t *__restrict__ out_hit, const int32_t *__restrict__ work,
                  int32_t *miss_list, int32_t *miss_rank) {
    __shared__ int warp_tot[32];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool miss = tid < B && out_hit[tid] == 0;
    const unsigned m = __ballot_sync(0xffffffffu, miss);
    if (lane == 0) warp_tot[warp] = __popc(m);
    __syncthreads();
    int base = 0;
    for (int w = 0; w < warp; ++w) base += warp_tot[w];
    if (miss) {
        const int rank = base + __popc(m & ((1u << lane) - 1u));
        miss_list[rank] = tid;
        miss_rank[tid] = rank;
    }
    if (tid == 0) {
        int n_miss = 0;
        for (int w = 0; w < 32; ++w) n_miss += warp_tot[w];
        st->n_miss = n_miss;
        st->n_risk = 0;
        st->count += n_miss - work[1];
        st->clock += B;
        st->queries += B;
        st->hits += B - n_miss;
        st->misses += n_miss;
        st->intra_hits += work[2];
        st->evictions += work[1];
    }
}

}  // namespace

void launch_lsh_probe(prox_handle *h, const float *q, int B, uint8_t *out_hit, cudaStream_t s) {
    lsh_hash_kernel<<<B, 256, 0, s>>>(B, h->d, h->lsh_L, q, h->planes, h->lsh_code);
    lsh_group_kernel<<<1, 1024, 0, s>>>(B, h->lsh_code, h->lsh_order, h->lsh_seg, h->lsh_work);
    lsh_resolve_kernel<<<B, 256, 0, s>>>(h->st, B, h->d, h->lsh_b, (double)h->tau, h->policy, q, h->lsh_code,
                                         h->lsh_order, h->lsh_seg, h->lsh_work, h->keys, h->stamp, h->bucket_count,
                                         out_hit, h->src, h->src_kind, h->ins_slot, h->evt_slot, h->evt_dist);
    lsh_finish_kernel<<<1, 1024, 0, s>>>(h->st, B, out_hit, h->lsh_work, h->miss_list, h->miss_rank);
    h->launches += 4;
}

}  // namespace prox
