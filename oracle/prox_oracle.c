/*
 * prox_oracle.c -- TEST INFRASTRUCTURE, not part of the product.
 *
 * A plain, slow, fp64 CPU statement of what the approximate query cache
 * computes, written from the paper so that the CUDA library can be checked
 * against it.  It shares no code with the CUDA path and must never be called
 * by it: only the tests, the smoke check and the CPU-baseline leg of the
 * benchmark may use it.
 *
 * What it follows:
 *   - Algorithm 1 ("Cache lookup in PROXIMITY-FLAT"), one query at a time, in
 *     stream order: distances from the query to every cached key, the nearest
 *     key, the test min_dist <= tau (inclusive, as Algorithm 1 and Section 3
 *     state it), the database call on a miss, eviction when |C| >= c, insert.
 *   - Section 3.3.2 (eviction policy): FIFO evicts the oldest inserted entry
 *     whatever its use; LRU evicts the entry unused for the longest time.
 *   - Section 2.2 (Vector search) / Section 3 (retrieveDocumentIndices): the database call is
 *     the exact k nearest rows of the corpus, returned as a list sorted by
 *     increasing distance (the FAISS-Flat case of Section 4.2.1).
 *
 * Readings where the paper is silent (the same readings are listed in the
 * design notes of the repository):
 *   - distance = squared Euclidean distance, for the cache keys and for the
 *     corpus alike (Section 3.1: the cache uses the database's distance);
 *   - ties between keys at equal distance go to the lowest slot; ties between
 *     corpus rows go to the lowest row id;
 *   - slots fill in index order 0..c-1, afterwards the victim's slot is reused;
 *   - every query owns one logical time stamp; an insert counts as a use;
 *   - a hit returns the stored list (and the stored distances of the key's own
 *     query) unchanged and alters nothing but the LRU stamp;
 *   - an empty cache is a miss; capacity 0 is rejected;
 *   - re-ranking factor rho (Section 3.3, "The re-ranking factor"): a miss asks the database for
 *     m = rho * k neighbours, stores all m under the key and returns the k nearest of them; a hit
 *     measures the m stored rows against the CURRENT query and returns the k nearest (distance
 *     ascending, ties to the lower row id) with those distances.  rho = 1 is "no re-ranking"
 *     (Section 4): the stored list comes back as it is, as above;
 *   - metric (Section 2.2, Vector search: the distance function is chosen once, before deployment):
 *     squared Euclidean by default; ORACLE_COSINE is the cosine distance 1 - cos(a, b), taken
 *     as half the squared Euclidean distance of a/|a| and b/|b| (the same number, and exactly 0
 *     for identical vectors so that tau = 0 stays exact matching); normalisation in fp64;
 *     ORACLE_IP is the inner product turned into a distance, -(a . b): the nearest key or row is
 *     the one with the largest inner product, and a key matches when -(q . key) <= tau, i.e. when
 *     q . key >= -tau.  For this metric tau may be any finite number (on unit vectors -1 <= -a.b
 *     <= 1), and tau = 0 is not exact matching: it accepts every key that is not on the far side
 *     of the query (inner product >= 0).  A vector is in general not its own nearest neighbour
 *     (a longer vector in the same direction scores higher);
 *   - PROXIMITY-LSH (Section 3.2): L random hyperplanes through the origin, given by the caller
 *     as L normal vectors; bit l of the hash is (q . r_l >= 0), the dot product taken in fp64
 *     in index order; the 2^L buckets are PROXIMITY-FLAT caches of b entries each, every one
 *     with its own FIFO / LRU eviction (Section 3.3.2, last sentence); bucket h owns the slots
 *     h*b .. h*b+b-1, filled in that order; time stamps stay global (one per query), which
 *     orders the entries of a bucket exactly as bucket-local stamps would.  Memory for all
 *     buckets is taken at once (the paper allocates a bucket at its first insert; the contents
 *     are the same).
 *
 * All sums are taken in double precision over the float inputs, one term
 * after the other in index order.  OpenMP only splits independent rows over
 * threads; the order inside a row and the selection pass stay sequential, so
 * the result does not depend on the thread count.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORACLE_LRU = 0, ORACLE_FIFO = 1 };
enum { ORACLE_L2SQ = 0, ORACLE_COSINE = 1, ORACLE_IP = 2 };

typedef struct {
    /* stored state of Algorithm 1: tau, c, the database D and the dict C */
    const float *corpus;   /* N x d, borrowed; NULL = trace-only (no database) */
    int64_t N;
    int32_t d, k;
    int32_t rho, m;        /* re-ranking factor and m = rho * k entries per value list */
    int32_t metric;        /* ORACLE_L2SQ or ORACLE_COSINE */
    int32_t lsh_L, lsh_b;  /* PROXIMITY-LSH: hyperplanes and bucket size; lsh_L < 0 = PROXIMITY-FLAT */
    float *planes;         /* lsh_L x d normal vectors (copy) */
    int64_t *bucket_count; /* 2^lsh_L */
    int64_t capacity;
    double tau;
    int32_t policy;
    /* the dict C: slot s holds a key (copy of the query), its value list */
    float *keys;           /* capacity x d */
    int64_t *val_ids;      /* capacity x m */
    double *val_dists;     /* capacity x m */
    int64_t *stamp;        /* capacity: LRU = last use, FIFO = insertion time */
    int64_t *origin;       /* capacity: stream index of the query that made the key */
    uint8_t *valid;        /* capacity */
    int64_t count;         /* |C| */
    int64_t clock;         /* logical time = number of queries seen */
    /* counters */
    int64_t probe_madds;   /* multiply-adds spent in key distances (Section 3.2: c*d per query) */
    int64_t n_hits, n_misses, n_evictions;
    double *scratch;       /* N distances for the database call */
} oracle_t;

int oracle_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* Threads that the row loops of the database call may use from now on (timing runs: one core, all cores). */
void oracle_set_threads(int n) {
#ifdef _OPENMP
    if (n >= 1) omp_set_num_threads(n);
#else
    (void)n;
#endif
}

/* Squared Euclidean distance, Algorithm 1 "distance(q, k)": sum_j (a_j - b_j)^2 in fp64. */
double oracle_sqdist(const float *a, const float *b, int32_t d) {
    double acc = 0.0;
    for (int32_t j = 0; j < d; ++j) {
        double diff = (double)a[j] - (double)b[j];
        acc += diff * diff;
    }
    return acc;
}

/* Cosine distance 1 - cos(a, b) = |a/|a| - b/|b||^2 / 2, every step in fp64. */
double oracle_cosdist(const float *a, const float *b, int32_t d) {
    double na = 0.0, nb = 0.0;
    for (int32_t j = 0; j < d; ++j) { na += (double)a[j] * (double)a[j]; nb += (double)b[j] * (double)b[j]; }
    na = sqrt(na); nb = sqrt(nb);
    double acc = 0.0;
    for (int32_t j = 0; j < d; ++j) {
        double diff = (double)a[j] / na - (double)b[j] / nb;
        acc += diff * diff;
    }
    return 0.5 * acc;
}

/* Inner product as a distance: -(a . b), the sum taken in fp64 in index order. */
double oracle_ipdist(const float *a, const float *b, int32_t d) {
    double acc = 0.0;
    for (int32_t j = 0; j < d; ++j) acc += (double)a[j] * (double)b[j];
    return -acc;
}

static double oracle_dist(int32_t metric, const float *a, const float *b, int32_t d) {
    if (metric == ORACLE_IP) return oracle_ipdist(a, b, d);
    return metric == ORACLE_COSINE ? oracle_cosdist(a, b, d) : oracle_sqdist(a, b, d);
}

/*
 * One pass of the selection behind retrieveDocumentIndices(q) over rows
 * [base_id, base_id + n) of the corpus (chunk points at row base_id).  The k
 * best rows seen so far are kept in out_ids / out_dists, sorted by (distance
 * ascending, row id ascending); *have is how many are filled.  Chunks must be
 * fed in ascending row order so that equal distances keep the lower id first.
 */
void oracle_topk_update_metric(int32_t metric, const float *chunk, int64_t n, int32_t d, int64_t base_id,
                               const float *q, int32_t k, double *scratch, int64_t *out_ids, double *out_dists,
                               int32_t *have_io) {
    double *dist = scratch;
    int own = 0;
    if (!dist) { dist = (double *)malloc(sizeof(double) * (size_t)n); own = 1; }
#pragma omp parallel for schedule(static)
    for (int64_t i = 0; i < n; ++i) dist[i] = oracle_dist(metric, q, chunk + i * (int64_t)d, d);

    int32_t have = *have_io;
    for (int64_t i = 0; i < n; ++i) {
        double v = dist[i];
        if (have == k && !(v < out_dists[k - 1])) continue;   /* equal to the worst: the earlier id stays */
        int32_t pos = (have < k) ? have : k - 1;
        while (pos > 0 && out_dists[pos - 1] > v) {            /* strictly greater: earlier ids stay in front */
            out_dists[pos] = out_dists[pos - 1];
            out_ids[pos] = out_ids[pos - 1];
            --pos;
        }
        out_dists[pos] = v;
        out_ids[pos] = base_id + i;
        if (have < k) ++have;
    }
    *have_io = have;
    if (own) free(dist);
}

void oracle_topk_update(const float *chunk, int64_t n, int32_t d, int64_t base_id, const float *q,
                        int32_t k, double *scratch, int64_t *out_ids, double *out_dists,
                        int32_t *have_io) {
    oracle_topk_update_metric(ORACLE_L2SQ, chunk, n, d, base_id, q, k, scratch, out_ids, out_dists, have_io);
}

/*
 * retrieveDocumentIndices(q): the k rows of the corpus closest to q, as a list
 * sorted by (distance ascending, row id ascending).  Every row is measured.
 */
void oracle_exact_topk_metric(int32_t metric, const float *corpus, int64_t N, int32_t d, const float *q, int32_t k,
                              double *scratch, int64_t *out_ids, double *out_dists) {
    int32_t have = 0;
    oracle_topk_update_metric(metric, corpus, N, d, 0, q, k, scratch, out_ids, out_dists, &have);
    for (int32_t r = have; r < k; ++r) { out_ids[r] = -1; out_dists[r] = INFINITY; }
}

void oracle_exact_topk(const float *corpus, int64_t N, int32_t d, const float *q, int32_t k,
                       double *scratch, int64_t *out_ids, double *out_dists) {
    oracle_exact_topk_metric(ORACLE_L2SQ, corpus, N, d, q, k, scratch, out_ids, out_dists);
}

oracle_t *oracle_create_rho(const float *corpus, int64_t N, int32_t d, int32_t k, int64_t capacity,
                            double tau, int32_t policy, int32_t rho) {
    if (d < 1 || k < 1 || capacity < 1 || rho < 1 || !(tau == tau) || isinf(tau)) return NULL;   /* the sign of tau: oracle_set_metric */
    if (policy != ORACLE_LRU && policy != ORACLE_FIFO) return NULL;
    const int32_t m = rho * k;
    if (corpus && (N < 1 || m > N)) return NULL;
    oracle_t *o = (oracle_t *)calloc(1, sizeof(oracle_t));
    if (!o) return NULL;
    o->corpus = corpus; o->N = N; o->d = d; o->k = k; o->rho = rho; o->m = m; o->lsh_L = -1;
    o->capacity = capacity; o->tau = tau; o->policy = policy;
    o->keys = (float *)calloc((size_t)capacity * d, sizeof(float));
    o->val_ids = (int64_t *)calloc((size_t)capacity * m, sizeof(int64_t));
    o->val_dists = (double *)calloc((size_t)capacity * m, sizeof(double));
    o->stamp = (int64_t *)calloc((size_t)capacity, sizeof(int64_t));
    o->origin = (int64_t *)calloc((size_t)capacity, sizeof(int64_t));
    o->valid = (uint8_t *)calloc((size_t)capacity, 1);
    o->scratch = corpus ? (double *)malloc(sizeof(double) * (size_t)N) : NULL;
    return o;
}

oracle_t *oracle_create(const float *corpus, int64_t N, int32_t d, int32_t k, int64_t capacity,
                        double tau, int32_t policy) {
    return oracle_create_rho(corpus, N, d, k, capacity, tau, policy, 1);
}

/* h(q) of Section 3.2: bit l = (q . r_l >= 0). */
int64_t oracle_lsh_hash(const float *planes, int32_t L, int32_t d, const float *q) {
    int64_t h = 0;
    for (int32_t l = 0; l < L; ++l) {
        double dot = 0.0;
        for (int32_t j = 0; j < d; ++j) dot += (double)q[j] * (double)planes[(int64_t)l * d + j];
        if (dot >= 0.0) h |= (int64_t)1 << l;
    }
    return h;
}

/* PROXIMITY-LSH: 2^L buckets of b entries; total capacity 2^L * b (Section 3.3.1). */
oracle_t *oracle_create_lsh(const float *corpus, int64_t N, int32_t d, int32_t k, int32_t L, int32_t b,
                            const float *planes, double tau, int32_t policy, int32_t rho) {
    if (L < 0 || L > 24 || b < 1 || (L > 0 && !planes)) return NULL;
    oracle_t *o = oracle_create_rho(corpus, N, d, k, ((int64_t)1 << L) * b, tau, policy, rho);
    if (!o) return NULL;
    o->lsh_L = L; o->lsh_b = b;
    o->planes = (float *)malloc(sizeof(float) * (size_t)(L > 0 ? L : 1) * d);
    if (L > 0) memcpy(o->planes, planes, sizeof(float) * (size_t)L * d);
    o->bucket_count = (int64_t *)calloc((size_t)1 << L, sizeof(int64_t));
    return o;
}

void oracle_destroy(oracle_t *o) {
    if (!o) return;
    free(o->planes); free(o->bucket_count);
    free(o->keys); free(o->val_ids); free(o->val_dists); free(o->stamp);
    free(o->origin); free(o->valid); free(o->scratch); free(o);
}

/* Chooses the distance of the cache keys and of the database (before the first query).  Squared
   Euclidean and cosine distances are never negative, so a negative tolerance is refused there;
   the inner-product distance takes any finite tolerance. */
int oracle_set_metric(oracle_t *o, int32_t metric) {
    if (metric != ORACLE_L2SQ && metric != ORACLE_COSINE && metric != ORACLE_IP) return 1;
    if (metric != ORACLE_IP && !(o->tau >= 0.0)) return 1;
    if (metric == ORACLE_IP && o->lsh_L >= 0) return 1;    /* hyperplane buckets go with angles, not with inner products */
    o->metric = metric;
    return 0;
}

void oracle_reset(oracle_t *o) {
    memset(o->valid, 0, (size_t)o->capacity);
    o->count = 0; o->clock = 0;
    if (o->bucket_count) memset(o->bucket_count, 0, sizeof(int64_t) << o->lsh_L);
    o->probe_madds = 0; o->n_hits = o->n_misses = o->n_evictions = 0;
}

void oracle_counters(const oracle_t *o, int64_t *out5) {
    out5[0] = o->probe_madds; out5[1] = o->n_hits; out5[2] = o->n_misses;
    out5[3] = o->n_evictions; out5[4] = o->count;
}

/* Load n keys into slots 0..n-1 with stamps 0..n-1 and empty value lists (test/bench set-up). */
int oracle_cache_load(oracle_t *o, const float *keys, int64_t n) {
    if (n < 0 || n > o->capacity) return 1;
    oracle_reset(o);
    memcpy(o->keys, keys, sizeof(float) * (size_t)n * o->d);
    for (int64_t s = 0; s < n; ++s) {
        o->valid[s] = 1; o->stamp[s] = s; o->origin[s] = -1 - s;
        for (int32_t r = 0; r < o->m; ++r) { o->val_ids[s * o->m + r] = -1; o->val_dists[s * o->m + r] = 0.0; }
    }
    o->count = n; o->clock = n;
    return 0;
}

/*
 * One LOOKUP(q) of Algorithm 1.
 *   force: -1 = decide by the threshold test; 0 / 1 = take "miss" / "hit"
 *          instead (used by a harness to keep two state machines in step on a
 *          query whose distance ties with tau to rounding; never by default).
 * Outputs (any may be NULL):
 *   out_ids[k], out_dists[k]  the returned list (dists: those stored with the key on a hit)
 *   trace[0] hit (0/1)
 *   trace[1] slot: the matched slot on a hit, the slot written on a miss
 *   trace[2] stream index of the query whose miss created the matched key (hit), else own index
 *   trace[3] slot evicted by this query, or -1
 *   dtrace[0] distance to the nearest key (+inf if the cache is empty)
 *   dtrace[1] distance to the second nearest key (+inf if fewer than two)
 */
void oracle_lookup(oracle_t *o, const float *q, int32_t force, int64_t *out_ids, double *out_dists,
                   int64_t *trace, double *dtrace) {
    const int32_t d = o->d, k = o->k, m = o->m;
    const int64_t t = o->clock++;                 /* this query's time stamp */

    /* Algorithm 1, the distances and their minimum: every valid key is measured, the first minimum in slot order wins */
    /* PROXIMITY-LSH: only the bucket that the hash names is looked at and updated */
    int64_t s_begin = 0, s_end = o->capacity, bucket = -1;
    if (o->lsh_L >= 0) {
        bucket = oracle_lsh_hash(o->planes, o->lsh_L, d, q);
        o->probe_madds += (int64_t)o->lsh_L * d;
        s_begin = bucket * o->lsh_b; s_end = s_begin + o->lsh_b;
    }
    double best = INFINITY, second = INFINITY;
    int64_t best_slot = -1;
    for (int64_t s = s_begin; s < s_end; ++s) {
        if (!o->valid[s]) continue;
        double dist = oracle_dist(o->metric, q, o->keys + s * d, d);
        o->probe_madds += d;
        if (dist < best) { second = best; best = dist; best_slot = s; }
        else if (dist < second) second = dist;
    }
    if (dtrace) { dtrace[0] = best; dtrace[1] = second; }

    int hit = (best_slot >= 0 && best <= o->tau);  /* the threshold test of Algorithm 1, inclusive */
    if (force == 0) hit = 0;
    if (force == 1 && best_slot >= 0) hit = 1;

    if (hit) {                                     /* hit: the value stored under the matched key */
        if (o->policy == ORACLE_LRU) o->stamp[best_slot] = t;   /* a hit is a use (LRU only) */
        const int64_t *sid = o->val_ids + best_slot * m;
        if (o->rho == 1 || !o->corpus) {           /* no re-ranking: the stored list, as it is */
            if (out_ids) memcpy(out_ids, sid, sizeof(int64_t) * k);
            if (out_dists) memcpy(out_dists, o->val_dists + best_slot * m, sizeof(double) * k);
        } else {
            /* re-ranking: the m stored rows measured against this query, the k nearest returned;
               insertion in (distance, row id) order, one stored row after the other */
            int64_t *rid = (int64_t *)malloc(sizeof(int64_t) * m);
            double *rd = (double *)malloc(sizeof(double) * m);
            int32_t have = 0;
            for (int32_t r = 0; r < m; ++r) {
                if (sid[r] < 0) continue;          /* the corpus had fewer than m rows */
                const double v = oracle_dist(o->metric, q, o->corpus + sid[r] * (int64_t)d, d);
                int32_t pos = have;
                while (pos > 0 && (rd[pos - 1] > v || (rd[pos - 1] == v && rid[pos - 1] > sid[r]))) {
                    rd[pos] = rd[pos - 1]; rid[pos] = rid[pos - 1]; --pos;
                }
                rd[pos] = v; rid[pos] = sid[r]; ++have;
            }
            for (int32_t r = 0; r < k; ++r) {
                if (out_ids) out_ids[r] = r < have ? rid[r] : -1;
                if (out_dists) out_dists[r] = r < have ? rd[r] : INFINITY;
            }
            free(rid); free(rd);
        }
        if (trace) { trace[0] = 1; trace[1] = best_slot; trace[2] = o->origin[best_slot]; trace[3] = -1; }
        o->n_hits++;
        return;
    }

    /* miss: the database is asked (retrieveDocumentIndices) */
    int64_t *ids = (int64_t *)malloc(sizeof(int64_t) * m);
    double *dists = (double *)malloc(sizeof(double) * m);
    if (o->corpus) oracle_exact_topk_metric(o->metric, o->corpus, o->N, d, q, m, o->scratch, ids, dists);   /* m = rho * k neighbours */
    else for (int32_t r = 0; r < m; ++r) { ids[r] = -1; dists[r] = 0.0; }

    /* a full cache (|C| >= c) gives up one entry first: the smallest stamp (stamps are unique) */
    int64_t slot, evicted = -1;
    const int64_t held = bucket >= 0 ? o->bucket_count[bucket] : o->count;      /* |C| of this (bucket's) cache */
    if (held >= s_end - s_begin) {
        slot = -1;
        for (int64_t s = s_begin; s < s_end; ++s)
            if (o->valid[s] && (slot < 0 || o->stamp[s] < o->stamp[slot])) slot = s;
        o->valid[slot] = 0; o->count--; o->n_evictions++;
        if (bucket >= 0) o->bucket_count[bucket]--;
        evicted = slot;
    } else {
        slot = s_begin + held;                     /* slots fill in index order */
    }

    /* the query becomes a key, the fetched list its value */
    memcpy(o->keys + slot * d, q, sizeof(float) * d);
    memcpy(o->val_ids + slot * m, ids, sizeof(int64_t) * m);
    memcpy(o->val_dists + slot * m, dists, sizeof(double) * m);
    o->valid[slot] = 1; o->stamp[slot] = t; o->origin[slot] = t; o->count++;
    if (bucket >= 0) o->bucket_count[bucket]++;
    o->n_misses++;

    /* the fetched list is returned (its k nearest when more were fetched) */
    if (out_ids) memcpy(out_ids, ids, sizeof(int64_t) * k);
    if (out_dists) memcpy(out_dists, dists, sizeof(double) * k);
    if (trace) { trace[0] = 0; trace[1] = slot; trace[2] = t; trace[3] = evicted; }
    free(ids); free(dists);
}

/* A stream of n queries, strictly one after the other.  force may be NULL. */
void oracle_query_stream(oracle_t *o, const float *queries, int64_t n, const int32_t *force,
                         int64_t *out_ids, double *out_dists, int64_t *trace, double *dtrace) {
    for (int64_t i = 0; i < n; ++i)
        oracle_lookup(o, queries + i * o->d, force ? force[i] : -1,
                      out_ids ? out_ids + i * o->k : NULL,
                      out_dists ? out_dists + i * o->k : NULL,
                      trace ? trace + i * 4 : NULL, dtrace ? dtrace + i * 2 : NULL);
}

/* The database call alone for a set of queries (used to check sampled misses at large N). */
void oracle_knn_batch_metric(int32_t metric, const float *corpus, int64_t N, int32_t d, const float *queries,
                             int64_t n, int32_t k, int64_t *out_ids, double *out_dists) {
    double *scratch = (double *)malloc(sizeof(double) * (size_t)N);
    for (int64_t i = 0; i < n; ++i)
        oracle_exact_topk_metric(metric, corpus, N, d, queries + i * d, k, scratch, out_ids + i * k, out_dists + i * k);
    free(scratch);
}

void oracle_knn_batch(const float *corpus, int64_t N, int32_t d, const float *queries, int64_t n,
                      int32_t k, int64_t *out_ids, double *out_dists) {
    oracle_knn_batch_metric(ORACLE_L2SQ, corpus, N, d, queries, n, k, out_ids, out_dists);
}

/* Read-only views for tests. */
int64_t oracle_slot_stamp(const oracle_t *o, int64_t s) { return o->valid[s] ? o->stamp[s] : -1; }
int64_t oracle_slot_origin(const oracle_t *o, int64_t s) { return o->valid[s] ? o->origin[s] : -1; }
