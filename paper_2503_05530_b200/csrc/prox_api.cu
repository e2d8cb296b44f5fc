// C ABI of the library: argument checks, memory, and the order of the kernels of one batch.
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "prox_internal.h"

using namespace prox;

static thread_local char g_err[256] = "";

namespace prox {
// Event pairs recorded around stage launches while prox_profile is on.
struct Profiler {
    struct Rec { cudaEvent_t a, b; int stage; };
    uint32_t mask = 0;
    std::vector<Rec> recs;      // used records
    std::vector<Rec> pool;      // events ready for reuse
    bool open_rec = false;
    void begin(int stage, cudaStream_t s) {
        if (!(mask >> stage & 1u)) return;
        Rec r;
        if (!pool.empty()) { r = pool.back(); pool.pop_back(); }
        else if (cudaEventCreate(&r.a) != cudaSuccess || cudaEventCreate(&r.b) != cudaSuccess) return;
        r.stage = stage;
        cudaEventRecord(r.a, s);
        recs.push_back(r);
        open_rec = true;
    }
    void end(cudaStream_t s) {
        if (open_rec) cudaEventRecord(recs.back().b, s);
        open_rec = false;
    }
    void drop() {
        for (auto &r : recs) pool.push_back(r);
        recs.clear();
    }
    ~Profiler() {
        drop();
        for (auto &r : pool) { cudaEventDestroy(r.a); cudaEventDestroy(r.b); }
    }
};
}  // namespace prox

struct StageScope {
    Profiler *p;
    cudaStream_t s;
    StageScope(prox_handle *h, int stage, cudaStream_t st) : p(h->prof), s(st) { if (p) p->begin(stage, s); }
    ~StageScope() { if (p) p->end(s); }
};

static void set_err(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}

extern "C" const char *prox_last_error(void) { return g_err; }

namespace prox {
// For entry points that live in other files: same thread-local text as set_err.
void set_last_error(const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
}
}  // namespace prox

template <typename T>
static bool dev_alloc(T *&p, size_t n) {
    void *q = nullptr;
    if (cudaMalloc(&q, n * sizeof(T)) != cudaSuccess) {
        cudaGetLastError();
        p = nullptr;
        return false;
    }
    p = static_cast<T *>(q);
    return true;
}

static void free_all(prox_handle *h) {
    void *ptrs[] = {h->over_list, h->over_d, h->over_id, h->over_ticket, h->redo, h->corpus_own, h->qn, h->planes, h->bucket_count, h->lsh_code, h->lsh_order, h->lsh_seg, h->lsh_work, h->xb, h->xh, h->keys, h->val_ids, h->val_dists, h->stamp, h->risk_pos, h->st,
                    h->risk_slot, h->risk_stamp, h->part_min, h->part_arg, h->d_risk, h->d_intra,
                    h->safe_min, h->safe_arg, h->cand_d, h->cand_code, h->n_cand, h->src, h->src_kind,
                    h->ins_slot, h->evt_slot, h->evt_dist, h->miss_list, h->miss_rank, h->qb, h->qbn,
                    h->qerr, h->thr_g, h->top1, h->buf, h->buf_cnt, h->cand_id, h->cand_score, h->cand_n,
                    h->cand_sk, h->res_ids, h->res_dists, h->fail_list, h->fail_radius, h->coll_id,
                    h->coll_n, h->stage_q, h->stage_ids, h->stage_dists, h->stage_hit, h->keys_b, h->kh, h->pqb,
                    h->pqbn, h->pqerr, h->use_partial, h->pfail_list, h->side_pairs};
    for (void *p : ptrs)
        if (p) cudaFree(p);
}

static int check_launch(const char *what) {
    const cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) {
        set_err("%s: %s", what, cudaGetErrorString(e));
        return PROX_ERR_CUDA;
    }
    return PROX_OK;
}

extern "C" prox_handle *prox_create(const float *corpus, int64_t N, int32_t d, int32_t k,
                                    int64_t capacity, float tau, int32_t policy) {
    return prox_create_rho(corpus, N, d, k, capacity, tau, policy, 1);
}

static prox_handle *create_handle(const float *corpus, int64_t N, int32_t d, int32_t k_out, int64_t capacity, float tau,
                                  int32_t policy, int32_t rho, int32_t metric);

extern "C" prox_handle *prox_create_rho(const float *corpus, int64_t N, int32_t d, int32_t k_out,
                                        int64_t capacity, float tau, int32_t policy, int32_t rho) {
    return create_handle(corpus, N, d, k_out, capacity, tau, policy, rho, PROX_METRIC_L2SQ);
}

// metric: PROX_METRIC_L2SQ (also the machinery under the cosine distance) or PROX_METRIC_IP.
static prox_handle *create_handle(const float *corpus, int64_t N, int32_t d, int32_t k_out, int64_t capacity, float tau,
                                  int32_t policy, int32_t rho, int32_t metric) {
    g_err[0] = 0;
    if (rho < 1) { set_err("rho must be >= 1"); return nullptr; }
    if (k_out < 1 || k_out > kMaxK || k_out > N) { set_err("k must be in [1, min(N, %d)]", kMaxK); return nullptr; }
    if ((long long)rho * k_out > kMaxFetch || (long long)rho * k_out > N) {
        set_err("rho * k must be at most min(N, %d)", kMaxFetch);
        return nullptr;
    }
    const int32_t k = rho * k_out;                        // entries fetched and stored per miss
    if (!corpus) { set_err("corpus is NULL"); return nullptr; }
    if (N < 1 || N >= (1LL << 31)) { set_err("N must be in [1, 2^31)"); return nullptr; }
    if (d < 16 || d > 4096 || d % 16) { set_err("d must be a multiple of 16 in [16, 4096]"); return nullptr; }
    if (capacity < 1 || capacity >= (1LL << 31)) { set_err("capacity must be in [1, 2^31)"); return nullptr; }
    if (metric == PROX_METRIC_IP) {
        if (std::isnan(tau) || std::isinf(tau)) { set_err("tau must be finite"); return nullptr; }
    } else if (!(tau >= 0.f) || std::isinf(tau)) {
        set_err("tau must be finite and >= 0");
        return nullptr;
    }
    if (policy != PROX_LRU && policy != PROX_FIFO) { set_err("policy must be PROX_LRU or PROX_FIFO"); return nullptr; }

    prox_handle *h = new (std::nothrow) prox_handle();
    if (!h) { set_err("out of host memory"); return nullptr; }
    std::memset(h, 0, sizeof(*h));
    h->corpus = corpus; h->N = N; h->d = d; h->k = k; h->k_out = k_out; h->rho = rho; h->lsh_L = -1; h->C = capacity; h->tau = tau; h->policy = policy; h->metric = metric;
    h->kp = 4 * k < 64 ? 64 : (4 * k > kMaxKp ? kMaxKp : 4 * k);
    h->scan_mode = PROX_SCAN_AUTO;
    cudaDeviceProp prop;
    if (cudaGetDevice(&h->device) != cudaSuccess ||
        cudaGetDeviceProperties(&prop, h->device) != cudaSuccess) {
        set_err("no CUDA device: %s", cudaGetErrorString(cudaGetLastError()));
        delete h;
        return nullptr;
    }
    if (prop.major != 10) {
        set_err("this library is built for sm_100a (B200); found compute capability %d.%d", prop.major, prop.minor);
        delete h;
        return nullptr;
    }
    h->num_sms = prop.multiProcessorCount;
    h->scan_ctas = h->num_sms;
    set_cache_kernel_attributes();
    set_probe_side_attributes();
    set_scan_kernel_attributes();

    const size_t MB = kMaxBatch, C = (size_t)capacity, P = (size_t)h->scan_ctas;
    bool ok = true;
    ok = ok && dev_alloc(h->xb, (size_t)N * d) && dev_alloc(h->xh, (size_t)N);
    ok = ok && dev_alloc(h->keys, C * d) && dev_alloc(h->val_ids, C * k) && dev_alloc(h->val_dists, C * k);
    ok = ok && dev_alloc(h->stamp, C) && dev_alloc(h->risk_pos, C) && dev_alloc(h->st, 1);
    ok = ok && dev_alloc(h->risk_slot, MB) && dev_alloc(h->risk_stamp, MB);
    ok = ok && dev_alloc(h->part_min, MB * kProbeSplitMax) && dev_alloc(h->part_arg, MB * kProbeSplitMax);
    ok = ok && dev_alloc(h->d_risk, MB * MB) && dev_alloc(h->d_intra, MB * MB);
    ok = ok && dev_alloc(h->safe_min, MB) && dev_alloc(h->safe_arg, MB);
    ok = ok && dev_alloc(h->cand_d, MB * 2 * MB) && dev_alloc(h->cand_code, MB * 2 * MB) && dev_alloc(h->n_cand, MB);
    ok = ok && dev_alloc(h->src, MB) && dev_alloc(h->src_kind, MB) && dev_alloc(h->ins_slot, MB);
    ok = ok && dev_alloc(h->evt_slot, MB) && dev_alloc(h->evt_dist, MB);
    ok = ok && dev_alloc(h->miss_list, MB) && dev_alloc(h->miss_rank, MB);
    ok = ok && dev_alloc(h->qb, MB * d) && dev_alloc(h->qbn, MB) && dev_alloc(h->qerr, MB) && dev_alloc(h->thr_g, MB);
    ok = ok && dev_alloc(h->top1, MB * 4 * P);          // per query: best score of every block's lane quarter
    h->tc_cap = h->kp <= 128 ? 256 : 512;               // four warp-private lists per block in the tensor-core scan
    // every pass of a batch (kScanQ queries each) keeps its lists until the one merge at the end
    constexpr size_t kPasses = kMaxBatch / kScanQ;
    h->buf_pass_stride = P * kScanQ * (size_t)(4 * h->tc_cap > kBufCap ? 4 * h->tc_cap : kBufCap);
    h->cnt_pass_stride = 4 * P * kScanQ;
    ok = ok && dev_alloc(h->buf, kPasses * h->buf_pass_stride) && dev_alloc(h->buf_cnt, kPasses * h->cnt_pass_stride);
    ok = ok && dev_alloc(h->cand_id, MB * kMaxKp) && dev_alloc(h->cand_score, MB * kMaxKp);
    ok = ok && dev_alloc(h->cand_n, MB) && dev_alloc(h->cand_sk, MB);
    ok = ok && dev_alloc(h->res_ids, MB * k) && dev_alloc(h->res_dists, MB * k);
    ok = ok && dev_alloc(h->fail_list, MB) && dev_alloc(h->fail_radius, MB);
    ok = ok && dev_alloc(h->coll_id, MB * kCollectCap) && dev_alloc(h->coll_n, MB) && dev_alloc(h->redo, MB + 1);
    ok = ok && dev_alloc(h->over_list, MB) && dev_alloc(h->over_d, (size_t)kOverMax * P * k) &&
         dev_alloc(h->over_id, (size_t)kOverMax * P * k) && dev_alloc(h->over_ticket, (size_t)kOverMax);
    // caches of a few thousand keys and more are probed on the tensor cores first (bf16 copies of the keys)
    // (the coarse probe's certificate is written for the Euclidean distance)
    h->probe_tc = (d % 64 == 0 && capacity >= 4096 && metric != PROX_METRIC_IP) ? 1 : 0;
    ok = ok && dev_alloc(h->use_partial, MB) && dev_alloc(h->pfail_list, MB);
    // bf16 copies of the keys and of the batch: for the coarse probe of large caches and for the
    // tensor-core pass over the at-risk slots and the batch itself (large batches)
    h->key_copies = metric != PROX_METRIC_IP ? 1 : 0;
    if (h->key_copies) {
        ok = ok && dev_alloc(h->keys_b, C * d) && dev_alloc(h->kh, C);
        ok = ok && dev_alloc(h->pqb, MB * d) && dev_alloc(h->pqbn, MB) && dev_alloc(h->pqerr, MB);
        ok = ok && dev_alloc(h->side_pairs, (size_t)kPairCap);
    }
    ok = ok && dev_alloc(h->stage_q, MB * d) && dev_alloc(h->stage_ids, MB * k);
    ok = ok && dev_alloc(h->stage_dists, MB * k) && dev_alloc(h->stage_hit, MB);
    if (!ok) {
        set_err("out of device memory");
        free_all(h);
        delete h;
        return nullptr;
    }
    cudaMemset(h->st, 0, sizeof(DevState));
    cudaMemset(h->qb, 0, MB * d * sizeof(__nv_bfloat16));
    if (h->key_copies) {
        cudaMemset(h->pqb, 0, MB * d * sizeof(__nv_bfloat16));
        cudaMemset(h->keys_b, 0, C * d * sizeof(__nv_bfloat16));
    }
    cudaMemset(h->buf_cnt, 0, kPasses * h->cnt_pass_stride * sizeof(int32_t));
    cudaMemset(h->over_ticket, 0, kOverMax * sizeof(unsigned));
    launch_convert_corpus(h, 0);
    launch_reset(h, 0);
    init_scan_tc(h);
    const cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) {
        set_err("set-up kernels failed: %s", cudaGetErrorString(e));
        free_all(h);
        delete h;
        return nullptr;
    }
    return h;
}

extern "C" prox_handle *prox_create_metric(const float *corpus, int64_t N, int32_t d, int32_t k, int64_t capacity,
                                           float tau, int32_t policy, int32_t rho, int32_t metric) {
    g_err[0] = 0;
    if (metric == PROX_METRIC_L2SQ) return prox_create_rho(corpus, N, d, k, capacity, tau, policy, rho);
    if (metric == PROX_METRIC_IP) return create_handle(corpus, N, d, k, capacity, tau, policy, rho, PROX_METRIC_IP);
    if (metric != PROX_METRIC_COSINE) { set_err("metric must be PROX_METRIC_L2SQ, PROX_METRIC_COSINE or PROX_METRIC_IP"); return nullptr; }
    if (!corpus) { set_err("corpus is NULL"); return nullptr; }
    if (N < 1 || N >= (1LL << 31) || d < 16 || d > 4096 || d % 16) { set_err("N or d out of range"); return nullptr; }
    if (!(tau >= 0.f) || std::isinf(tau)) { set_err("tau must be finite and >= 0"); return nullptr; }
    // 1 - cos(a, b) = |a/|a| - b/|b||^2 / 2: the Euclidean machinery on unit-length copies, at 2 tau
    float *own = nullptr, *qn = nullptr;
    if (!dev_alloc(own, (size_t)N * d) || !dev_alloc(qn, (size_t)kMaxBatch * d)) {
        set_err("out of device memory for the unit-length copy of the corpus");
        if (own) cudaFree(own);
        return nullptr;
    }
    launch_normalize_rows(corpus, own, N, d, 0);
    prox_handle *h = prox_create_rho(own, N, d, k, capacity, 2.f * tau, policy, rho);
    if (!h) {
        cudaFree(own);
        cudaFree(qn);
        return nullptr;
    }
    h->metric = PROX_METRIC_COSINE; h->corpus_own = own; h->qn = qn;
    return h;
}

extern "C" prox_handle *prox_create_lsh(const float *corpus, int64_t N, int32_t d, int32_t k, int32_t L, int32_t b,
                                        const float *planes, float tau, int32_t policy, int32_t rho) {
    g_err[0] = 0;
    if (L < 0 || L > 20) { set_err("L must be in [0, 20]"); return nullptr; }
    if (b < 1 || b > 64) { set_err("the bucket size b must be in [1, 64]"); return nullptr; }
    if (L > 0 && !planes) { set_err("planes is NULL"); return nullptr; }
    if (((int64_t)b << L) >= (1LL << 31)) { set_err("2^L * b must be below 2^31"); return nullptr; }
    prox_handle *h = prox_create_rho(corpus, N, d, k, (int64_t)b << L, tau, policy, rho);
    if (!h) return nullptr;
    h->lsh_L = L; h->lsh_b = b;
    h->probe_tc = 0; h->key_copies = 0;                   // buckets are probed directly; no bf16 key copies are kept
    const size_t MB = kMaxBatch;
    bool ok = dev_alloc(h->planes, (size_t)(L > 0 ? L : 1) * d) && dev_alloc(h->bucket_count, (size_t)1 << L) &&
              dev_alloc(h->lsh_code, MB) && dev_alloc(h->lsh_order, MB) && dev_alloc(h->lsh_seg, MB + 1) &&
              dev_alloc(h->lsh_work, 4);
    if (ok) {
        if (L > 0) cudaMemcpy(h->planes, planes, (size_t)L * d * sizeof(float), cudaMemcpyDeviceToDevice);
        cudaMemset(h->bucket_count, 0, sizeof(int32_t) << L);
        ok = cudaDeviceSynchronize() == cudaSuccess;
    }
    if (!ok) {
        set_err("out of device memory for the buckets: %s", cudaGetErrorString(cudaGetLastError()));
        free_all(h);
        delete h;
        return nullptr;
    }
    return h;
}

extern "C" void prox_destroy(prox_handle *h) {
    if (!h) return;
    cudaDeviceSynchronize();
    delete h->prof;
    free_scan_tc(h);
    free_all(h);
    delete h;
}

static int check_batch_args(prox_handle *h, const void *queries, int32_t B) {
    g_err[0] = 0;
    if (!h) { set_err("handle is NULL"); return PROX_ERR_INVALID_ARG; }
    if (!queries) { set_err("queries is NULL"); return PROX_ERR_INVALID_ARG; }
    if (B < 1 || B > kMaxBatch) { set_err("B must be in [1, %d]", kMaxBatch); return PROX_ERR_INVALID_ARG; }
    return PROX_OK;
}

// gather_ids / gather_dists: where the stored lists of hits on pre-batch keys may be copied to in
// the same pass (NULL: the caller does it).  Returns true when that copy has been done.
static bool enqueue_probe_and_resolve(prox_handle *h, const float *queries, int32_t B, uint8_t *out_hit,
                                      int64_t *gather_ids, float *gather_dists, cudaStream_t s) {
    if (h->lsh_L >= 0) {                                  // PROXIMITY-LSH: the query's bucket only
        StageScope t(h, PROX_STAGE_PROBE, s);
        launch_lsh_probe(h, queries, B, out_hit, s);
        return false;
    }
    if (small_lookup_fits(h, B) && h->scan_mode != PROX_SCAN_CUDA_CORE) {   // a few queries, a small cache: two launches
        StageScope t(h, PROX_STAGE_PROBE, s);
        launch_small_lookup(h, queries, B, out_hit, gather_ids, gather_dists, s);
        return gather_ids != nullptr;
    }
    { StageScope t(h, PROX_STAGE_RISK_SELECT, s); launch_risk_select(h, B, s); }
    // large batches: the at-risk slots and the batch itself on the tensor cores, exact recheck of the
    // pairs that could lie within tau (instead of B x 2B fp64 rows)
    const bool side = h->key_copies && h->scan_mode != PROX_SCAN_CUDA_CORE && B >= kSideMinBatch;
    int splits = -1;
    {
        StageScope t(h, PROX_STAGE_PROBE, s);
        // the coarse pass has a fixed cost of a few launches: it pays off from about two million
        // query-key pairs per batch on
        bool coarse = h->probe_tc && h->scan_mode != PROX_SCAN_CUDA_CORE && (long long)B * h->C >= 2LL * (1 << 20);
        if (coarse || side) launch_prep_probe(h, queries, B, s);
        if (coarse) {
            // safe slots: coarse scores on the tensor cores, exact recheck of the best few;
            // at-risk slots and the batch itself: full fp64 rows (or the pass above); uncertified
            // queries: fp64 over all slots
            if (launch_probe_scan_tc(h, B, s) != 0) coarse = false;
            if (coarse) launch_merge_select(h, B, 1, s);
        }
        if (side) launch_probe_side(h, queries, B, s);
        if (coarse) {
            launch_probe_exact(h, queries, B, s);
            launch_probe(h, queries, B, side ? 4 : 1, s);
            launch_probe(h, queries, B, 2, s);
        } else {
            if (h->probe_tc) cudaMemsetAsync(h->use_partial, 0xff, sizeof(int32_t) * kMaxBatch, s);   // all from partials
            if (side) {
                // a capacity within the batch size: every stored key is at risk, there is no safe slot to scan
                if (h->C > B) launch_probe(h, queries, B, 3, s);
                else splits = 0;
                launch_probe(h, queries, B, 4, s);
            } else {
                launch_probe(h, queries, B, 0, s);
            }
        }
    }
    { StageScope t(h, PROX_STAGE_CANDIDATES, s); launch_build_candidates(h, B, splits, side ? 1 : 0, s); }
    { StageScope t(h, PROX_STAGE_RESOLVE, s); launch_resolve(h, B, out_hit, s); }
    return false;
}

// First half of a batch: probe and replay, answers of hits on stored keys, and for every miss
// the exact k nearest rows of the corpus held here (res_ids / res_dists).  Returns the queries
// the rest of the batch works on (unit-length copies for the cosine distance).
static const float *enqueue_lookup_and_scan(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                                            float *out_dists, uint8_t *out_hit, cudaStream_t s) {
    if (h->metric == PROX_METRIC_COSINE) {                // unit-length copies stand in for the queries from here on
        launch_normalize_rows(queries, h->qn, B, h->d, s);
        h->launches++;
        queries = h->qn;
    }

    const bool gathered = enqueue_probe_and_resolve(h, queries, B, out_hit, h->rho == 1 ? out_ids : nullptr,
                                                    h->rho == 1 ? out_dists : nullptr, s);
    if (!gathered) {
        StageScope t(h, PROX_STAGE_GATHER, s);
        if (h->rho == 1) launch_gather_hits(h, B, out_ids, out_dists, s);
        else launch_hit_rerank(h, queries, B, 1, out_ids, out_dists, s);     // before the scatter rewrites slots
    }
    if (small_corpus_fits(h, B) && h->scan_mode == PROX_SCAN_AUTO) {
        StageScope t(h, PROX_STAGE_SCAN, s);
        launch_small_exact(h, queries, s);
        return queries;
    }
    { StageScope t(h, PROX_STAGE_PREP_MISS, s); launch_prep_miss(h, queries, B, s); }
    const int passes = (B + kScanQ - 1) / kScanQ;
    {
        StageScope t(h, PROX_STAGE_SCAN, s);
        // the tensor-core scan takes all passes of the batch in one launch, its CUDA-core twin one by one
        if (h->scan_mode == PROX_SCAN_CUDA_CORE || launch_scan_tc(h, B, s) != 0)
            for (int p = 0; p < passes; ++p) launch_scan_pass(h, p, s);
    }
    { StageScope t(h, PROX_STAGE_MERGE, s); launch_merge_select(h, B, 0, s); }
    { StageScope t(h, PROX_STAGE_RERANK, s); launch_rerank(h, queries, B, s); }
    { StageScope t(h, PROX_STAGE_EXACT_PASS, s); launch_fallback(h, queries, B, s); }
    return queries;
}

// Second half: answers of the misses and of the hits on keys of this batch, insertion of the
// batch's new keys with their lists (from res_ids / res_dists).
static void enqueue_answers_and_inserts(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                                        float *out_dists, cudaStream_t s) {
    {
        StageScope t(h, PROX_STAGE_SCATTER, s);
        if (h->rho > 1) launch_hit_rerank(h, queries, B, 2, out_ids, out_dists, s);   // hits on keys of this batch
        launch_scatter(h, queries, B, out_ids, out_dists, 1, s);
    }
    if (h->metric == PROX_METRIC_COSINE) {                // squared distance of unit vectors -> 1 - cos
        launch_scale(out_dists, (long long)B * h->k_out, 0.5f, s);
        h->launches++;
    }
}

extern "C" int32_t prox_query_batch(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                                    float *out_dists, uint8_t *out_hit, void *stream) {
    int rc = check_batch_args(h, queries, B);
    if (rc) return rc;
    if (!out_ids || !out_dists || !out_hit) { set_err("an output pointer is NULL"); return PROX_ERR_INVALID_ARG; }
    if (h->sharded) {
        set_err("this handle holds one shard of a corpus: use prox_shard_scan and prox_shard_merge");
        return PROX_ERR_INVALID_ARG;
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    queries = enqueue_lookup_and_scan(h, queries, B, out_ids, out_dists, out_hit, s);
    enqueue_answers_and_inserts(h, queries, B, out_ids, out_dists, s);
    return check_launch("prox_query_batch");
}

// ------------------------------------------------------------------------------------------
// A batch call recorded once and replayed: the launches of prox_query_batch with fixed buffers,
// captured into a CUDA graph.  For small batches over small corpora the device work of a batch is
// tens of microseconds and the chain of launches is what a call costs; a replay submits the
// whole chain with one call.  Two recordings are kept, because consecutive scans alternate the
// halves of the pairs' speed table: the replays alternate the same way.
// ------------------------------------------------------------------------------------------
struct prox_recorded_batch {
    prox_handle *h;
    cudaGraphExec_t exec[2];
    int64_t launches_per_call;
    unsigned turn;
};

extern "C" prox_recorded_batch *prox_record_batch(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                                                  float *out_dists, uint8_t *out_hit, void *stream) {
    if (check_batch_args(h, queries, B)) return nullptr;
    if (!out_ids || !out_dists || !out_hit) { set_err("an output pointer is NULL"); return nullptr; }
    if (h->sharded) { set_err("a shard's calls are not recorded"); return nullptr; }
    if (h->prof) { set_err("switch prox_profile off before recording: its events would become part of the recording"); return nullptr; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    prox_recorded_batch *r = new (std::nothrow) prox_recorded_batch();
    if (!r) { set_err("out of host memory"); return nullptr; }
    r->h = h; r->exec[0] = r->exec[1] = nullptr; r->turn = 0;
    const int64_t launches0 = h->launches;
    for (int i = 0; i < 2; ++i) {
        cudaGraph_t g = nullptr;
        cudaError_t e = cudaStreamBeginCapture(s, cudaStreamCaptureModeThreadLocal);
        if (e == cudaSuccess) {
            const float *q = enqueue_lookup_and_scan(h, queries, B, out_ids, out_dists, out_hit, s);
            enqueue_answers_and_inserts(h, q, B, out_ids, out_dists, s);
            e = cudaStreamEndCapture(s, &g);
        }
        if (e == cudaSuccess) e = cudaGraphInstantiate(&r->exec[i], g, 0);
        if (g) cudaGraphDestroy(g);
        if (e != cudaSuccess) {
            set_err("prox_record_batch: %s", cudaGetErrorString(e));
            cudaGetLastError();
            if (r->exec[0]) cudaGraphExecDestroy(r->exec[0]);
            delete r;
            h->launches = launches0;
            return nullptr;
        }
    }
    r->launches_per_call = (h->launches - launches0) / 2;
    h->launches = launches0;                                  // nothing has run yet
    return r;
}

extern "C" int32_t prox_replay_batch(prox_recorded_batch *r, void *stream) {
    g_err[0] = 0;
    if (!r) { set_err("recording is NULL"); return PROX_ERR_INVALID_ARG; }
    const cudaError_t e = cudaGraphLaunch(r->exec[r->turn & 1u], static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        set_err("prox_replay_batch: %s", cudaGetErrorString(e));
        cudaGetLastError();
        return PROX_ERR_CUDA;
    }
    r->turn++;
    r->h->launches += r->launches_per_call;
    return PROX_OK;
}

extern "C" void prox_recorded_batch_destroy(prox_recorded_batch *r) {
    if (!r) return;
    for (int i = 0; i < 2; ++i)
        if (r->exec[i]) cudaGraphExecDestroy(r->exec[i]);
    delete r;
}

extern "C" prox_handle *prox_create_shard(const float *corpus, int64_t N, int32_t d, int32_t k, int64_t capacity,
                                          float tau, int32_t policy, int32_t metric, int64_t row_offset,
                                          int64_t n_total) {
    g_err[0] = 0;
    if (n_total < 1 || n_total >= (1LL << 31)) { set_err("n_total must be in [1, 2^31)"); return nullptr; }
    if (row_offset < 0 || N < 1 || row_offset > n_total - N) {
        set_err("the shard's rows [row_offset, row_offset + N) must lie within [0, n_total)");
        return nullptr;
    }
    prox_handle *h = prox_create_metric(corpus, N, d, k, capacity, tau, policy, 1, metric);
    if (!h) return nullptr;
    h->sharded = 1; h->row_offset = row_offset; h->n_total = n_total;
    return h;
}

extern "C" int64_t prox_shard_exchange_bytes(const prox_handle *h, int32_t B) {
    if (!h || B < 1 || B > kMaxBatch) return 0;
    return (int64_t)16 * B * h->k;
}

extern "C" int32_t prox_shard_scan(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                                   float *out_dists, uint8_t *out_hit, void *xchg, void *stream) {
    int rc = check_batch_args(h, queries, B);
    if (rc) return rc;
    if (!out_ids || !out_dists || !out_hit || !xchg) { set_err("an output pointer is NULL"); return PROX_ERR_INVALID_ARG; }
    if (!h->sharded) { set_err("not a shard handle (prox_create_shard)"); return PROX_ERR_INVALID_ARG; }
    if (reinterpret_cast<uintptr_t>(xchg) % 16) { set_err("xchg must be 16-byte aligned"); return PROX_ERR_INVALID_ARG; }
    if (h->shard_pending) { set_err("the previous prox_shard_scan was not completed by prox_shard_merge"); return PROX_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    enqueue_lookup_and_scan(h, queries, B, out_ids, out_dists, out_hit, s);
    { StageScope t(h, PROX_STAGE_SCATTER, s); launch_shard_pack(h, B, xchg, s); }
    h->shard_pending = B;
    return check_launch("prox_shard_scan");
}

extern "C" int32_t prox_shard_merge(prox_handle *h, const float *queries, int32_t B, const void *gathered, int32_t G,
                                    int64_t *out_ids, float *out_dists, void *stream) {
    int rc = check_batch_args(h, queries, B);
    if (rc) return rc;
    if (!out_ids || !out_dists || !gathered) { set_err("a pointer is NULL"); return PROX_ERR_INVALID_ARG; }
    if (!h->sharded) { set_err("not a shard handle (prox_create_shard)"); return PROX_ERR_INVALID_ARG; }
    if (G < 1 || G > 32) { set_err("G must be in [1, 32]"); return PROX_ERR_INVALID_ARG; }
    if (reinterpret_cast<uintptr_t>(gathered) % 16) { set_err("gathered must be 16-byte aligned"); return PROX_ERR_INVALID_ARG; }
    if (h->shard_pending != B) { set_err("no prox_shard_scan of %d queries is waiting for its merge", B); return PROX_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (h->metric == PROX_METRIC_COSINE) queries = h->qn;  // the unit-length copies made by prox_shard_scan
    { StageScope t(h, PROX_STAGE_MERGE, s); launch_shard_merge(h, B, gathered, G, s); }
    enqueue_answers_and_inserts(h, queries, B, out_ids, out_dists, s);
    h->shard_pending = 0;
    return check_launch("prox_shard_merge");
}

extern "C" int32_t prox_query_batch_host(prox_handle *h, const float *queries, int32_t B, int64_t *out_ids,
                                         float *out_dists, uint8_t *out_hit, void *stream) {
    int rc = check_batch_args(h, queries, B);
    if (rc) return rc;
    if (!out_ids || !out_dists || !out_hit) { set_err("an output pointer is NULL"); return PROX_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const size_t k = h->k_out;
    if (cudaMemcpyAsync(h->stage_q, queries, (size_t)B * h->d * sizeof(float), cudaMemcpyHostToDevice, s) !=
        cudaSuccess)
        return check_launch("copy of the queries");
    rc = prox_query_batch(h, h->stage_q, B, h->stage_ids, h->stage_dists, h->stage_hit, stream);
    if (rc) return rc;
    cudaMemcpyAsync(out_ids, h->stage_ids, (size_t)B * k * sizeof(int64_t), cudaMemcpyDeviceToHost, s);
    cudaMemcpyAsync(out_dists, h->stage_dists, (size_t)B * k * sizeof(float), cudaMemcpyDeviceToHost, s);
    cudaMemcpyAsync(out_hit, h->stage_hit, (size_t)B, cudaMemcpyDeviceToHost, s);
    const cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) {
        set_err("prox_query_batch_host: %s", cudaGetErrorString(e));
        return PROX_ERR_CUDA;
    }
    return PROX_OK;
}

extern "C" int32_t prox_probe_batch(prox_handle *h, const float *queries, int32_t B, uint8_t *out_hit,
                                    int32_t *out_slot, float *out_min_dist, void *stream) {
    int rc = check_batch_args(h, queries, B);
    if (rc) return rc;
    if (!out_hit) { set_err("out_hit is NULL"); return PROX_ERR_INVALID_ARG; }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    if (h->metric == PROX_METRIC_COSINE) {
        launch_normalize_rows(queries, h->qn, B, h->d, s);
        h->launches++;
        queries = h->qn;
    }
    enqueue_probe_and_resolve(h, queries, B, out_hit, nullptr, nullptr, s);
    if (out_slot || out_min_dist) launch_probe_outputs(h, B, out_slot, out_min_dist, s);
    if (out_min_dist && h->metric == PROX_METRIC_COSINE) {
        launch_scale(out_min_dist, B, 0.5f, s);
        h->launches++;
    }
    { StageScope t(h, PROX_STAGE_SCATTER, s); launch_scatter(h, queries, B, nullptr, nullptr, 0, s); }
    return check_launch("prox_probe_batch");
}

extern "C" int32_t prox_reset_cache(prox_handle *h, void *stream) {
    g_err[0] = 0;
    if (!h) { set_err("handle is NULL"); return PROX_ERR_INVALID_ARG; }
    launch_reset(h, static_cast<cudaStream_t>(stream));
    h->shard_pending = 0;
    if (h->lsh_L >= 0) cudaMemsetAsync(h->bucket_count, 0, sizeof(int32_t) << h->lsh_L, static_cast<cudaStream_t>(stream));
    return check_launch("prox_reset_cache");
}

extern "C" int32_t prox_cache_load(prox_handle *h, const float *keys, int64_t n, void *stream) {
    g_err[0] = 0;
    if (!h) { set_err("handle is NULL"); return PROX_ERR_INVALID_ARG; }
    if (n < 0 || n > h->C) { set_err("n must be in [0, capacity]"); return PROX_ERR_INVALID_ARG; }
    if (n > 0 && !keys) { set_err("keys is NULL"); return PROX_ERR_INVALID_ARG; }
    if (h->lsh_L >= 0) { set_err("prox_cache_load is not available for a PROXIMITY-LSH handle"); return PROX_ERR_UNSUPPORTED; }
    if (h->metric == PROX_METRIC_COSINE && n > 0) {       // the keys are stored at unit length
        launch_normalize_rows(keys, h->keys, n, h->d, static_cast<cudaStream_t>(stream));
        h->launches++;
        keys = h->keys;
    }
    launch_cache_load(h, keys, n, static_cast<cudaStream_t>(stream));
    return check_launch("prox_cache_load");
}

extern "C" int32_t prox_get_stats(prox_handle *h, prox_stats *out, void *stream) {
    g_err[0] = 0;
    if (!h || !out) { set_err("NULL argument"); return PROX_ERR_INVALID_ARG; }
    DevState st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(&st, h->st, sizeof(st), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { set_err("prox_get_stats: %s", cudaGetErrorString(e)); return PROX_ERR_CUDA; }
    out->queries = st.queries; out->hits = st.hits; out->misses = st.misses;
    out->intra_batch_hits = st.intra_hits; out->evictions = st.evictions;
    out->scan_batches = st.scan_batches; out->uncertified = st.uncertified;
    out->fallback_rows = st.fallback_rows; out->unresolved = st.unresolved; out->count = st.count;
    out->probe_uncertified = st.probe_uncertified;
    out->parallel_replays = st.parallel_replays;
    return PROX_OK;
}

extern "C" int32_t prox_status(prox_handle *h, void *stream) {
    g_err[0] = 0;
    if (!h) { set_err("handle is NULL"); return PROX_ERR_INVALID_ARG; }
    DevState st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(&st, h->st, sizeof(st), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) { set_err("prox_status: %s", cudaGetErrorString(e)); return PROX_ERR_CUDA; }
    if (st.error) set_err("device-side error %d latched", st.error);
    return st.error;
}

extern "C" int32_t prox_set_scan_mode(prox_handle *h, int32_t mode) {
    g_err[0] = 0;
    if (!h || (mode != PROX_SCAN_AUTO && mode != PROX_SCAN_CUDA_CORE && mode != PROX_SCAN_TC_SINGLE)) {
        set_err("bad handle or mode");
        return PROX_ERR_INVALID_ARG;
    }
    h->scan_mode = mode;
    return PROX_OK;
}

extern "C" int64_t prox_kernel_launches(const prox_handle *h) { return h ? h->launches : 0; }

extern "C" int32_t prox_profile(prox_handle *h, uint32_t stage_mask) {
    g_err[0] = 0;
    if (!h) { set_err("handle is NULL"); return PROX_ERR_INVALID_ARG; }
    if (stage_mask == 0) {
        delete h->prof;
        h->prof = nullptr;
        return PROX_OK;
    }
    if (!h->prof) h->prof = new (std::nothrow) Profiler();
    if (!h->prof) { set_err("out of host memory"); return PROX_ERR_OOM; }
    h->prof->mask = stage_mask;
    return PROX_OK;
}

extern "C" int32_t prox_profile_read(prox_handle *h, double *ms_by_stage, int64_t *launches_by_stage,
                                     void *stream) {
    g_err[0] = 0;
    if (!h || !ms_by_stage || !launches_by_stage) { set_err("NULL argument"); return PROX_ERR_INVALID_ARG; }
    for (int i = 0; i < PROX_N_STAGES; ++i) { ms_by_stage[i] = 0.0; launches_by_stage[i] = 0; }
    const cudaError_t e = cudaStreamSynchronize(static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) { set_err("prox_profile_read: %s", cudaGetErrorString(e)); return PROX_ERR_CUDA; }
    if (!h->prof) return PROX_OK;
    for (auto &r : h->prof->recs) {
        float ms = 0.f;
        if (cudaEventElapsedTime(&ms, r.a, r.b) == cudaSuccess) {
            ms_by_stage[r.stage] += ms;
            launches_by_stage[r.stage] += 1;
        } else {
            cudaGetLastError();
        }
    }
    h->prof->drop();
    return PROX_OK;
}
