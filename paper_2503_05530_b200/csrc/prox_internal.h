// Internal layout of a handle and the host-side launchers of every kernel.
#pragma once
#include <cstdint>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "../../include/prox.h"

namespace prox {

constexpr int kMaxK = PROX_MAX_K;            // largest k
constexpr int kMaxFetch = PROX_MAX_FETCH;    // largest rho * k
constexpr int kMaxKp = 256;                  // largest k' (candidates kept by the coarse scan)
constexpr int kMaxBatch = PROX_MAX_BATCH;    // largest B
constexpr int kScanQ = 256;                  // queries per scan pass (MMA N dimension)
constexpr int kTileRows = 128;               // corpus rows per scan tile (MMA M dimension)
constexpr int kBufCap = 512;                 // entries of one (CTA, query) candidate buffer
constexpr int kCollectCap = 2048;            // rows the exact pass may collect per query
constexpr int kOverMax = 64;                 // queries per batch whose collection may overflow and still be answered exactly
constexpr int kProbeSplitMax = 128;          // column splits of the probe grid
constexpr int kPairCap = 1 << 20;             // query-key pairs the tensor-core pass over at-risk slots and batch may hand on
constexpr int kSideMinBatch = 512;            // batches from this size on take that pass instead of fp64 rows
constexpr int kProbeKp = 64;                 // slots per query the coarse probe keeps for the exact recheck

// Device-resident scalars of a handle.
struct DevState {
    long long count;          // |C|
    long long clock;          // logical time = queries seen (plus loaded keys)
    int n_risk;               // at-risk slots of the current batch
    int n_miss;               // misses of the current batch
    int n_fail;               // misses whose candidate set was not certified
    int error;                // latched PROX_ERR_* found on the device
    float e_max;              // upper bound of |x - bf16(x)| over corpus rows
    float xn_max;             // upper bound of |bf16(x)| over corpus rows
    float ke_max;             // upper bound of |key - bf16(key)| over the keys inserted since the last reset
    float kn_max;             // upper bound of |bf16(key)| over those keys
    int n_probe;              // queries of the current batch (read by the coarse probe's kernels)
    int n_pfail;              // queries whose coarse probe was not certified
    int n_over;               // queries whose exact pass collected more rows than it can hold
    long long stamp_floor;    // a lower bound of every stored stamp (the smallest stamp of the last at-risk selection)
    long long fifo_head;      // FIFO: slot of the oldest entry (the stored entries form a ring in slot order)
    int n_pairs;              // pairs listed by the tensor-core pass over the at-risk slots and the batch
    int side_overflow;        // 1 = more such pairs than the list holds: the fp64 rows are used instead
    // statistics
    long long queries, hits, misses, intra_hits, evictions, scan_batches, uncertified,
        fallback_rows, unresolved, probe_uncertified, parallel_replays;
};

struct Profiler;

}  // namespace prox

struct prox_handle {
    // stored state of Algorithm 1
    const float *corpus;      // N x d fp32, borrowed
    int64_t N;
    int32_t d, k, kp;         // k: entries of a value list (rho * k_out)
    int32_t k_out, rho;       // neighbours returned per query; re-ranking factor
    // cosine distance: own unit-length copy of the corpus, unit-length copies of the batch queries
    int32_t metric;
    float *corpus_own;        // N x d (NULL for the Euclidean distance)
    float *qn;                // kMaxBatch x d
    // PROXIMITY-LSH (lsh_L < 0: flat cache)
    int32_t lsh_L, lsh_b;
    float *planes;            // lsh_L x d normal vectors
    int32_t *bucket_count;    // 2^lsh_L: entries held by each bucket
    int32_t *lsh_code;        // kMaxBatch: bucket of each batch query
    int32_t *lsh_order;       // kMaxBatch: batch queries sorted by (bucket, index)
    int32_t *lsh_seg;         // kMaxBatch + 1: where each bucket's run starts in lsh_order
    int32_t *lsh_work;        // [0] number of runs, [1] evictions, [2] hits on keys of this batch
    // a corpus split by rows over several GPUs (sharded = 0: the whole corpus is here)
    int32_t sharded;
    int64_t row_offset;       // id of this shard's first row
    int64_t n_total;          // rows of the whole corpus
    int32_t shard_pending;    // batch size of a prox_shard_scan that prox_shard_merge has not completed, else 0
    int64_t C;
    float tau;
    int32_t policy;
    int device, num_sms;
    int scan_mode;
    int64_t launches;
    prox::Profiler *prof;     // event records of prox_profile (NULL when off)
    void *tc_state;           // tensor maps of the tensor-core scan (made on first use)

    // corpus copies for the scan
    __nv_bfloat16 *xb;        // N x d
    float *xh;                // N: 0.5 * |bf16(x)|^2

    // key-value store
    float *keys;              // C x d
    int32_t *val_ids;         // C x k
    float *val_dists;         // C x k
    unsigned long long *stamp;  // C
    int32_t *risk_pos;        // C: position in the at-risk list or -1
    __nv_bfloat16 *keys_b;    // C x d: bf16 copies of the keys for the tensor-core probe
    float *kh;                // C: 0.5 * |bf16(key)|^2, +inf for an empty slot
    prox::DevState *st;

    // per-batch scratch
    int32_t *risk_slot;               // kMaxBatch
    unsigned long long *risk_stamp;   // kMaxBatch
    double *part_min;                 // kMaxBatch x kProbeSplitMax
    int32_t *part_arg;                // kMaxBatch x kProbeSplitMax
    double *d_risk;                   // kMaxBatch x kMaxBatch
    double *d_intra;                  // kMaxBatch x kMaxBatch
    double *safe_min;                 // kMaxBatch
    int32_t *safe_arg;                // kMaxBatch
    double *cand_d;                   // kMaxBatch x 2 kMaxBatch   (probe candidates <= tau)
    int32_t *cand_code;               // kMaxBatch x 2 kMaxBatch
    int32_t *n_cand;                  // kMaxBatch
    int32_t *src;                     // kMaxBatch: hit source (slot, or batch index), -1 on a miss
    int32_t *src_kind;                // kMaxBatch: 0 miss, 1 pre-batch slot, 2 batch entry
    int32_t *ins_slot;                // kMaxBatch: slot written at batch end or -1
    int32_t *evt_slot;                // kMaxBatch: matched / written slot at the time of the lookup
    float *evt_dist;                  // kMaxBatch: distance to the matched key (+inf on a miss)
    __nv_bfloat16 *pqb;               // kMaxBatch x d: bf16 copies of all batch queries (coarse probe)
    float *pqbn;                      // kMaxBatch: |bf16(q)|^2
    float *pqerr;                     // kMaxBatch: upper bound of |q - bf16(q)|
    int32_t *use_partial;             // kMaxBatch: 1 = the safe minimum comes from the fp64 probe's partial minima
    int32_t *pfail_list;              // kMaxBatch: queries that take the exact fp64 probe
    int32_t probe_tc;                 // 1 = coarse tensor-core probe in use for this handle
    int32_t key_copies;               // 1 = bf16 copies of the keys are kept (coarse probe, tensor-core pass over at-risk slots)
    uint32_t *side_pairs;             // kPairCap: (query << 16 | code) of the pairs that pass
    void *tc_state_keys;              // tensor maps of the coarse probe
    int32_t *miss_list;               // kMaxBatch
    int32_t *miss_rank;               // kMaxBatch

    __nv_bfloat16 *qb;                // kMaxBatch x d: bf16 copies of the miss queries
    float *qbn;                       // kMaxBatch: |bf16(q)|^2
    float *qerr;                      // kMaxBatch: upper bound of |q - bf16(q)|
    uint32_t *thr_g;                  // kMaxBatch: shared score thresholds (ordered-uint form)
    uint32_t *top1;                   // kMaxBatch x P: each block's best score per miss query (ordered-uint form)
    unsigned long long *buf;          // candidate lists of the scan blocks (layout set by the scan that ran)
    int32_t *buf_cnt;                 // entries per list
    int32_t scan_ctas;                // P
    size_t buf_pass_stride;           // entries of `buf` that one scan pass (up to kScanQ queries) owns
    size_t cnt_pass_stride;           // entries of `buf_cnt` that one scan pass owns
    int32_t scan_lists;               // lists per query written by the last scan pass
    int32_t scan_list_stride;         // entries between consecutive (list, query) buffers
    int32_t tc_cap;                   // entries per (warp, query) buffer of the tensor-core scan
    int32_t *cand_id;                 // kMaxBatch x kMaxKp
    float *cand_score;                // kMaxBatch x kMaxKp
    int32_t *cand_n;                  // kMaxBatch
    float *cand_sk;                   // kMaxBatch: k'-th best coarse score (-inf if fewer rows)
    int32_t *res_ids;                 // kMaxBatch x k
    double *res_dists;                // kMaxBatch x k
    int32_t *fail_list;               // kMaxBatch
    float *fail_radius;               // kMaxBatch: exact k-th distance among the candidates
    int32_t *coll_id;                 // kMaxBatch x kCollectCap (indexed by position in fail_list)
    int32_t *coll_n;                  // kMaxBatch
    int32_t *redo;                    // kMaxBatch + 1: queries the fp32 sweep of the exact pass takes again; [kMaxBatch] any
    int32_t *over_list;               // kMaxBatch: places in fail_list of the queries whose collection overflowed
    double *over_d;                   // kOverMax x blocks x k: every block's nearest rows of its share of the corpus
    int32_t *over_id;                 // kOverMax x blocks x k
    unsigned *over_ticket;            // kOverMax: blocks that have delivered their list (back to 0 after the merge)

    // staging for the host-buffer entry point
    float *stage_q;
    int64_t *stage_ids;
    float *stage_dists;
    uint8_t *stage_hit;
};

namespace prox {
// per-device kernel attributes (dynamic shared memory limits), set at prox_create
void set_cache_kernel_attributes();
void set_probe_side_attributes();
void set_scan_kernel_attributes();
// create-time kernels
void launch_convert_corpus(prox_handle *h, cudaStream_t s);
inline bool metric_is_ip(const prox_handle *h) { return h->metric == PROX_METRIC_IP; }
// cache kernels
void launch_risk_select(prox_handle *h, int B, cudaStream_t s);
void launch_probe(prox_handle *h, const float *q, int B, int mode, cudaStream_t s);   // 0 all slots + batch, 1 at-risk + batch, 2 failed queries, 3 safe slots only, 4 = 1 if the pair list overflowed
void launch_build_candidates(prox_handle *h, int B, int splits, int lists_ready, cudaStream_t s);   // splits < 0: as the probe used
void launch_resolve(prox_handle *h, int B, uint8_t *out_hit, cudaStream_t s);
void launch_gather_hits(prox_handle *h, int B, int64_t *out_ids, float *out_dists, cudaStream_t s);
bool small_lookup_fits(const prox_handle *h, int B);
void launch_small_lookup(prox_handle *h, const float *q, int B, uint8_t *out_hit, int64_t *out_ids, float *out_dists,
                         cudaStream_t s);   // small B and capacity: probe .. replay (.. gather when out_ids is given) in two launches
void launch_hit_rerank(prox_handle *h, const float *q, int B, int kind, int64_t *out_ids, float *out_dists,
                       cudaStream_t s);   // rho > 1: hits of that kind (1 stored key, 2 key of this batch)
void launch_scatter(prox_handle *h, const float *q, int B, int64_t *out_ids, float *out_dists,
                    int with_values, cudaStream_t s);
void launch_normalize_rows(const float *src, float *dst, long long n, int d, cudaStream_t s);   // dst = src / |src| per row (may alias)
void launch_scale(float *v, long long n, float f, cudaStream_t s);
void launch_lsh_probe(prox_handle *h, const float *q, int B, uint8_t *out_hit, cudaStream_t s);   // hash, group, replay per bucket
void launch_probe_outputs(prox_handle *h, int B, int32_t *out_slot, float *out_min_dist, cudaStream_t s);
void launch_cache_load(prox_handle *h, const float *keys, int64_t n, cudaStream_t s);
void launch_reset(prox_handle *h, cudaStream_t s);
// scan kernels
void launch_prep_miss(prox_handle *h, const float *q, int B, cudaStream_t s);
void launch_prep_probe(prox_handle *h, const float *q, int B, cudaStream_t s);
int launch_probe_scan_tc(prox_handle *h, int B, cudaStream_t s);              // coarse probe over the bf16 keys, all passes; nonzero = not available
void launch_probe_exact(prox_handle *h, const float *q, int B, cudaStream_t s);
void launch_probe_side(prox_handle *h, const float *q, int B, cudaStream_t s);   // at-risk slots and batch on the tensor cores -> candidate lists
void launch_scan_pass(prox_handle *h, int pass, cudaStream_t s);       // CUDA-core scan
int launch_scan_tc(prox_handle *h, int B, cudaStream_t s);                  // tcgen05 scan, all passes of the batch; nonzero = not available
void init_scan_tc(prox_handle *h);                                      // tensor maps, at prox_create
void free_scan_tc(prox_handle *h);
void launch_merge_select(prox_handle *h, int B, int for_probe, cudaStream_t s);   // all passes of the batch at once
void launch_rerank(prox_handle *h, const float *q, int B, cudaStream_t s);
void launch_fallback(prox_handle *h, const float *q, int B, cudaStream_t s);
bool small_corpus_fits(const prox_handle *h, int B);
void launch_small_exact(prox_handle *h, const float *q, cudaStream_t s);   // all misses of a small batch over a small corpus, fp64, one launch
// row shards
void launch_shard_pack(prox_handle *h, int B, void *xchg, cudaStream_t s);       // this shard's exchange record
void launch_shard_merge(prox_handle *h, int B, const void *gathered, int G, cudaStream_t s);   // G records -> res_ids / res_dists
}  // namespace prox
