/*
 * prox.h -- C ABI of the B200 approximate query cache with exact top-k corpus scan.
 *
 * The library keeps, on one GPU, the state of Algorithm 1 of the paper ("Cache
 * lookup in PROXIMITY-FLAT"): the tolerance tau, the capacity c, the database D
 * (a corpus of N embeddings of dimension d) and the key-value store C whose keys
 * are earlier query embeddings and whose values are their top-k lists.  One call
 * of prox_query_batch performs LOOKUP(q) for a batch of queries with exactly the
 * outcome of running Algorithm 1 on them one after the other in index order.
 *
 * Conventions
 *  - Distances are squared Euclidean distances, for keys and corpus alike
 *    (Section 3.1: the cache uses the distance function of the database), unless the
 *    handle was made by prox_create_metric with the cosine distance or the inner product.
 *  - Every pointer marked DEVICE is a device pointer valid on the GPU that was
 *    current when prox_create ran; HOST pointers are ordinary host memory.
 *  - Calls on one handle must be ordered on one stream at a time: the cache is
 *    state.  prox_query_batch only enqueues work; its outputs are valid once
 *    the stream has reached the end of that work.
 *  - Functions returning int32_t return PROX_OK or an error code; a text for the
 *    last error of the calling thread is available from prox_last_error().
 *  - Inputs must be finite; this is not checked on the device.
 */
#ifndef PROX_H_
#define PROX_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct prox_handle prox_handle;      /* opaque, owned by the library */

enum { PROX_LRU = 0, PROX_FIFO = 1 };        /* Section 3.3.2: eviction policy */

enum {
    PROX_OK = 0,
    PROX_ERR_INVALID_ARG = 1,   /* nothing was launched */
    PROX_ERR_OOM = 2,
    PROX_ERR_CUDA = 3,
    PROX_ERR_UNSUPPORTED = 4,   /* shape outside what the kernels are built for */
    PROX_ERR_TIMEOUT = 5,       /* a bounded device-side wait ran out (latched) */
    PROX_ERR_INTERNAL = 6       /* a device-side capacity or bounds check failed (latched) */
};

enum {
    PROX_MAX_K = 64,            /* largest k */
    PROX_MAX_FETCH = 128,       /* largest rho * k (neighbours fetched and stored per miss) */
    PROX_MAX_BATCH = 1024,      /* largest B of one call */
    PROX_METRIC_L2SQ = 0,       /* prox_create_metric: squared Euclidean distance (the default everywhere else) */
    PROX_METRIC_COSINE = 1,     /* prox_create_metric: cosine distance 1 - cos(a, b) */
    PROX_METRIC_IP = 2,         /* prox_create_metric: inner product as a distance, -(a . b) */
    PROX_SCAN_AUTO = 0,         /* prox_set_scan_mode: tensor-core scan, two blocks per MMA (default) */
    PROX_SCAN_CUDA_CORE = 1,    /* prox_set_scan_mode: plain CUDA-core scan of the same bf16 scores */
    PROX_SCAN_TC_SINGLE = 2     /* prox_set_scan_mode: tensor-core scan, one block per MMA */
};

/*
 * prox_create -- set up the stored state of Algorithm 1 (tau, c, D, C = {}).
 *   corpus   DEVICE, N x d fp32 row-major, BORROWED: the caller keeps it alive and
 *            unchanged until prox_destroy.  The library makes its own bf16 copy
 *            (round to nearest even) and per-row norms for the scan.
 *   N        number of corpus rows, 1 <= N < 2^31.
 *   d        embedding dimension, a multiple of 16, 16 <= d <= 4096.
 *   k        neighbours per query, 1 <= k <= min(N, PROX_MAX_K).
 *   capacity c of Section 3.3.1, >= 1 (c = 0 is rejected: Algorithm 1 would evict from an empty store).
 *   tau      tolerance of Section 3.3.3 on the squared distance, >= 0 and not NaN;
 *            a key matches when distance <= tau (the threshold test of Algorithm 1).
 *   policy   PROX_LRU or PROX_FIFO.
 * Returns NULL on failure (see prox_last_error).  Allocates with cudaMalloc on
 * the current device and synchronises that device before returning.
 */
prox_handle *prox_create(const float *corpus, int64_t N, int32_t d, int32_t k, int64_t capacity,
                         float tau, int32_t policy);

/*
 * prox_create_rho -- prox_create with the re-ranking factor rho >= 1 of Section 3.3
 * ("The re-ranking factor"): a miss fetches the rho * k nearest corpus rows, stores all of
 * them under the key and returns the k nearest; a hit measures the rho * k stored rows
 * against the CURRENT query (exact squared distances) and returns the k nearest of them,
 * nearest first, ties by lower id, with those distances.  rho = 1 is prox_create: no
 * re-ranking, the stored list comes back as it is.  rho * k <= min(N, PROX_MAX_FETCH).
 */
prox_handle *prox_create_rho(const float *corpus, int64_t N, int32_t d, int32_t k, int64_t capacity,
                             float tau, int32_t policy, int32_t rho);

/*
 * prox_create_metric -- prox_create_rho with the distance named (Section 2.2, Vector search: the
 * distance function is chosen once, before deployment; Section 3.1: the cache uses the
 * database's distance).  PROX_METRIC_COSINE: keys and corpus rows are compared by
 * 1 - cos(a, b), evaluated as half the squared Euclidean distance of a/|a| and b/|b| (identical
 * vectors, of any length, are at distance exactly 0); tau applies to that value and out_dists
 * hold it.  The library keeps its own unit-length fp32 copy of the corpus (N x d x 4 bytes
 * more) and brings every query to unit length (norms in fp64) before the lookup.  Rows and
 * queries must be non-zero.
 * PROX_METRIC_IP: the inner product turned into a distance, -(a . b): the nearest key or row is
 * the one with the largest inner product with the query, a key matches when -(q . key) <= tau
 * (q . key >= -tau), and out_dists hold -(q . row), most similar first.  For this metric tau may
 * be any finite number, negative ones included (on unit vectors the value lies in [-1, 1]); tau = 0
 * is not exact matching here, it accepts every key whose inner product with the query is >= 0,
 * and a query is in general not its own nearest key (a longer key in the same direction scores
 * higher).  Not offered for PROXIMITY-LSH handles; large caches are probed in fp64 only.
 */
prox_handle *prox_create_metric(const float *corpus, int64_t N, int32_t d, int32_t k, int64_t capacity,
                                float tau, int32_t policy, int32_t rho, int32_t metric);

/*
 * prox_create_lsh -- PROXIMITY-LSH of Section 3.2: the cache is split into 2^L buckets of b
 * entries; a query is looked up in, and on a miss inserted into, the one bucket that its hash
 * h(q) = (q . r_1 >= 0, ..., q . r_L >= 0) names (bit l-1 of the bucket number belongs to r_l;
 * dot products in fp64).  Every bucket is a PROXIMITY-FLAT cache with its own FIFO / LRU
 * eviction (Section 3.3.2); bucket h owns the slots h*b .. h*b+b-1.  Total capacity 2^L * b.
 *   planes   DEVICE, L x d fp32 row-major: the hyperplanes' normal vectors r_1..r_L, drawn by
 *            the caller (the library draws no random numbers); copied.  May be NULL when L = 0.
 *   L        0 <= L <= 20 (L = 0: one bucket, i.e. a flat cache of b entries).
 *   b        bucket size, 1 <= b <= 64 (the paper uses 20), 2^L * b < 2^31.
 *   rho      re-ranking factor as in prox_create_rho (1 = none).
 * All buckets are allocated at once (the paper allocates a bucket at its first insert; with
 * the memory of this GPU the difference is moot).  prox_cache_load is not available for such
 * a handle.  Everything else (prox_query_batch, prox_probe_batch, ...) works as for a flat cache.
 */
prox_handle *prox_create_lsh(const float *corpus, int64_t N, int32_t d, int32_t k, int32_t L, int32_t b,
                             const float *planes, float tau, int32_t policy, int32_t rho);

/*
 * prox_query_batch -- LOOKUP(q) of Algorithm 1 for queries 0..B-1, with the
 * outcome of processing them strictly in index order: query i sees the inserts,
 * evictions and LRU touches of queries 0..i-1 of the same batch.
 *   queries   DEVICE, B x d fp32 row-major, borrowed until the enqueued work is done.
 *   B         1 <= B <= PROX_MAX_BATCH.
 *   out_ids   DEVICE, B x k int64: the returned list I (corpus row ids, nearest first;
 *             ties by lower id).  On a hit: the list stored with the matched key.
 *   out_dists DEVICE, B x k fp32: squared distances belonging to out_ids.  On a hit these
 *             are the distances stored with the key, i.e. those of the key's own query.
 *             (With rho > 1, see prox_create_rho: a hit returns the k stored rows nearest
 *             to this query with their distances to this query.)
 *   out_hit   DEVICE, B bytes: 1 = cache hit (the stored list is returned), 0 = miss (the database is asked and the result inserted).
 *   stream    a cudaStream_t (NULL = the default stream).
 * Misses are answered by an exact k-nearest-neighbour search over the whole corpus
 * (the database call of Algorithm 1, with a flat exact index as in Section 4.2.1).
 * Asynchronous; no device-to-host copy and no synchronisation happens inside.
 * Errors found on the device are latched and reported by prox_status.
 */
int32_t prox_query_batch(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                         float *out_dists, uint8_t *out_hit, void *stream);

/*
 * prox_query_batch_host -- the same call for HOST buffers (queries, out_ids, out_dists,
 * out_hit are host pointers, ideally pinned).  Copies the queries to the device, runs
 * prox_query_batch, copies the three outputs back and synchronises the stream.
 */
int32_t prox_query_batch_host(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                              float *out_dists, uint8_t *out_hit, void *stream);

/* ---- a corpus split by rows over several GPUs -------------------------------------------- */

/*
 * The database call of Algorithm 1 over a corpus too large for one GPU; the paper
 * has no counterpart of this split, it is an addition of this library.  GPU g of G holds the
 * rows [row_offset, row_offset + N) of the corpus; the cache and the queries are replicated:
 * every GPU runs the same lookup on the same queries, so the G caches stay equal without any
 * exchange.  Only the miss path differs: each GPU finds the k nearest rows of ITS shard
 * (prox_shard_scan), the G lists of every miss are brought to every GPU by the caller (one
 * all-gather of prox_shard_exchange_bytes bytes per GPU, any transport), and each GPU merges
 * them into the k nearest of the whole corpus (prox_shard_merge; ties by lower id, so all GPUs
 * arrive at the same bytes).  Row ids everywhere are ids of the whole corpus.
 *
 * prox_create_shard -- as prox_create_metric with rho = 1, for one shard.
 *   corpus      DEVICE, N x d fp32: the shard's rows, borrowed.
 *   N           rows of this shard, k <= N.
 *   row_offset  id of the shard's first row; row_offset + N <= n_total.
 *   n_total     rows of the whole corpus, < 2^31.
 * A shard handle answers through prox_shard_scan / prox_shard_merge; prox_query_batch and
 * prox_query_batch_host reject it.  prox_probe_batch, prox_cache_load, prox_reset_cache and the
 * diagnostics work as usual.
 */
prox_handle *prox_create_shard(const float *corpus, int64_t N, int32_t d, int32_t k, int64_t capacity,
                               float tau, int32_t policy, int32_t metric, int64_t row_offset,
                               int64_t n_total);

/*
 * prox_shard_exchange_bytes -- size of one GPU's exchange record for a batch of B queries:
 * B * k fp64 distances followed by B * k int64 row ids (16 * B * k bytes), miss j of the batch
 * (in index order) at entries j*k .. j*k+k-1; the entries of places beyond the batch's number
 * of misses hold distance +inf and id -1.  0 if an argument is out of range.
 */
int64_t prox_shard_exchange_bytes(const prox_handle *h, int32_t B);

/*
 * prox_shard_scan -- first half of LOOKUP for a batch: probe, threshold test, replay of the
 * batch (hit flags, evictions, slots), the answers of hits on stored keys, and the exact k
 * nearest rows of this shard for every miss.
 *   queries, B, out_ids, out_dists, out_hit, stream: as in prox_query_batch; after this call
 *             out_hit is final, out_ids / out_dists are final for hits on stored keys only.
 *   xchg      DEVICE, prox_shard_exchange_bytes(h, B) bytes, 16-byte aligned: this GPU's record.
 * Asynchronous.  Must be followed by prox_shard_merge for the same batch before the next batch.
 */
int32_t prox_shard_scan(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                        float *out_dists, uint8_t *out_hit, void *xchg, void *stream);

/*
 * prox_shard_merge -- second half: merges the G records, writes the answers of the misses and
 * of the hits on keys of this batch, and inserts the batch's new keys with their lists.
 *   gathered  DEVICE, G records back to back (any order of shards; every shard exactly once).
 *   G         number of shards, 1 <= G <= 32.
 *   queries, B, out_ids, out_dists: the arguments of the prox_shard_scan call this completes.
 * Asynchronous.
 */
int32_t prox_shard_merge(prox_handle *h, const float *queries, int32_t B, const void *gathered, int32_t G,
                         int64_t *out_ids, float *out_dists, void *stream);

/*
 * prox_record_batch -- records the launches of one prox_query_batch call with these buffers as a CUDA graph and
 * returns a handle for replaying it; nothing runs yet and the cache is not touched.  A replay is one such call
 * on whatever the buffers hold at that time (same B, same addresses), with the launches submitted in one go: for
 * small batches over small corpora, where a call costs its chain of launches rather than its device work (the
 * sequential use of Algorithm 1, one query at a time), a replay is 10-20 % faster than the call.  Results, cache
 * state and counters are those of prox_query_batch.  Rules: all five pointers DEVICE and valid for every replay;
 * prox_profile off while recording; `stream` must not be the legacy default stream (stream capture) and is left as
 * it was; replays of one recording and other calls on the handle are ordered by the caller (one stream, or events),
 * as for every entry point.  A recording belongs to its handle: destroy it before prox_destroy.  Not for shards.
 * Returns NULL on error (prox_last_error()).
 */
typedef struct prox_recorded_batch prox_recorded_batch;
prox_recorded_batch *prox_record_batch(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                                       float *out_dists, uint8_t *out_hit, void *stream);

/* prox_replay_batch -- enqueues one recorded batch on `stream` (asynchronous). */
int32_t prox_replay_batch(prox_recorded_batch *r, void *stream);

/* prox_recorded_batch_destroy -- frees the recording (not the handle). NULL is allowed. */
void prox_recorded_batch_destroy(prox_recorded_batch *r);

/* prox_reset_cache -- C = {} (count and clock to zero); the corpus stays.  Asynchronous on stream. */
int32_t prox_reset_cache(prox_handle *h, void *stream);

/* prox_destroy -- synchronise the device and free everything the library owns.  NULL is a no-op. */
void prox_destroy(prox_handle *h);

/* prox_last_error -- text of the calling thread's last error ("" if none); static storage. */
const char *prox_last_error(void);

/* ---- diagnostics and benchmark hooks (outside Algorithm 1) ------------------------------- */

/*
 * prox_cache_load -- fill slots 0..n-1 with the given keys (DEVICE, n x d fp32), stamps
 * 0..n-1 and empty value lists (ids -1, distances 0); count = clock = n.  Stands in for
 * n earlier misses when only the probe is measured (the lookup-time experiment of
 * Section 4.5.1, lookup times for increasing cache occupancies).  n <= capacity.  Asynchronous on stream.
 */
int32_t prox_cache_load(prox_handle *h, const float *keys, int64_t n, void *stream);

/*
 * prox_probe_batch -- Algorithm 1 without its database call: probe, threshold test,
 * LRU touch, eviction and insertion of the query as a key, with an empty value list in
 * place of the database call.
 *   out_hit      DEVICE, B bytes.
 *   out_slot     DEVICE, B int32: the matched slot on a hit, the written slot on a miss.
 *   out_min_dist DEVICE, B fp32: on a hit the distance to the matched (nearest) key, on a miss +inf.
 */
int32_t prox_probe_batch(prox_handle *h, const float *queries, int32_t B, uint8_t *out_hit,
                         int32_t *out_slot, float *out_min_dist, void *stream);

typedef struct prox_stats {
    int64_t queries, hits, misses;      /* since create / reset */
    int64_t intra_batch_hits;           /* hits on a key inserted earlier in the same batch */
    int64_t evictions;
    int64_t scan_batches;               /* batches in which the corpus was scanned */
    int64_t uncertified;                /* misses whose bf16 candidate set was not proven complete */
    int64_t fallback_rows;              /* rows collected by the exact fp32 pass for those misses */
    int64_t unresolved;                 /* misses whose exact pass overflowed (result best effort) */
    int64_t count;                      /* |C| now */
    int64_t probe_uncertified;          /* queries whose coarse (tensor-core) probe fell back to the exact fp64 probe */
    int64_t parallel_replays;           /* batches whose replay was solved as a fixed point instead of in query order */
} prox_stats;

/* prox_get_stats -- synchronises the stream, then copies the device counters to *out (HOST). */
int32_t prox_get_stats(prox_handle *h, prox_stats *out, void *stream);

/* prox_status -- synchronises the stream and returns the latched device error (PROX_OK if none). */
int32_t prox_status(prox_handle *h, void *stream);

/* prox_set_scan_mode -- one of the PROX_SCAN_* values (for cross-checks and timing). */
int32_t prox_set_scan_mode(prox_handle *h, int32_t mode);

/* prox_kernel_launches -- kernels launched by this handle so far (host-side count). */
int64_t prox_kernel_launches(const prox_handle *h);

/* Stages of one batch, in launch order (indices of the arrays of prox_profile_read).  A batch of up to four
 * queries against a small cache runs its whole lookup (at-risk selection to gather) under PROX_STAGE_PROBE, and
 * over a small corpus its whole database call (scan to exact pass) under PROX_STAGE_SCAN. */
enum {
    PROX_STAGE_RISK_SELECT = 0, PROX_STAGE_PROBE = 1, PROX_STAGE_CANDIDATES = 2, PROX_STAGE_RESOLVE = 3,
    PROX_STAGE_GATHER = 4, PROX_STAGE_PREP_MISS = 5, PROX_STAGE_SCAN = 6, PROX_STAGE_MERGE = 7,
    PROX_STAGE_RERANK = 8, PROX_STAGE_EXACT_PASS = 9, PROX_STAGE_SCATTER = 10, PROX_N_STAGES = 11
};

/*
 * prox_profile -- stage_mask bit s set: record a pair of CUDA events on the caller's stream
 * around every launch of stage s from now on (0 switches recording off and drops what was
 * recorded).  For measurement only: each pair costs about a microsecond of stream time.
 */
int32_t prox_profile(prox_handle *h, uint32_t stage_mask);

/*
 * prox_profile_read -- synchronises the stream, adds up the recorded intervals per stage into
 * ms_by_stage[PROX_N_STAGES] and their number into launches_by_stage[PROX_N_STAGES] (both HOST),
 * and clears the records.  A stage launched for a batch without misses still counts: its
 * kernels return at once.
 */
int32_t prox_profile_read(prox_handle *h, double *ms_by_stage, int64_t *launches_by_stage, void *stream);

/* ---- a lookup for callers that must not allocate ------------------------------------------ */

enum {
    PROX_STATIC_MAX_BATCH = 256,        /* largest B of prox_nearest_key_static */
    PROX_STATIC_MAX_KEYS = 1 << 22      /* largest n_keys of prox_nearest_key_static */
};

/*
 * prox_nearest_key_static -- for every query the nearest of n_keys keys and its squared distance
 * (the paper has no counterpart of this entry point, it is an addition of this library).  It is meant for callers that cannot allocate device memory at
 * the time of the call: code embedded in an application that owns all GPU memory and forbids
 * further allocations, code running with a fixed memory budget, a thread that must not touch the
 * allocator.  The call needs no handle, calls no cudaMalloc / cudaFree and no allocating library
 * routine; the partial results its blocks exchange live in an array of about 192 KB that is part
 * of the library image on every GPU that loads it, until the process exits.
 *   keys      DEVICE, n_keys x d fp32 row-major, 1 <= n_keys <= PROX_STATIC_MAX_KEYS, 1 <= d <= 4096.
 *   queries   DEVICE, B x d fp32 row-major, 1 <= B <= PROX_STATIC_MAX_BATCH.
 *   out_slot  DEVICE, B int32: row of the nearest key (lowest row on a tie).
 *   out_dist  DEVICE, B fp32: its squared distance (fp64 sum over the fp32 values, rounded once).
 * Sizes beyond these limits are rejected with PROX_ERR_INVALID_ARG and a text in prox_last_error();
 * nothing is launched then.  Asynchronous on stream.
 * The first call on a GPU looks up the device address of the built-in array (once per GPU, with
 * that GPU current); make that first call outside any stream capture.  The address is kept for
 * the life of the process: it does not survive a cudaDeviceReset of that GPU, after which this
 * entry point must not be called again in the same process.
 * All calls on one GPU share the array, which keeps the last call's contents (the call clears the
 * counters it needs at zero itself): calls that could run at the same time on one GPU race with
 * each other, so order them on one stream.
 */
int32_t prox_nearest_key_static(const float *keys, int64_t n_keys, int32_t d, const float *queries, int32_t B,
                                int32_t *out_slot, float *out_dist, void *stream);

#ifdef __cplusplus
}
#endif
#endif /* PROX_H_ */
