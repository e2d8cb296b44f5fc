"""GPU parity: the CUDA library, called through its C ABI, against the fp64 oracle on the same
seeded bytes, element by element."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05530_b200 import prox, workloads as W
from golden_traces import all_load_traces, all_traces
import oracle_workers
import parity
from parity import compare, run_gpu, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def stream(N, d, comps, nq, topics, s, sigma, seed=0):
    X = W.make_corpus(N, d, comps, seed)
    Q, _, _ = W.make_query_stream(X, nq, topics, s, sigma, seed)
    return X, Q


def check(X, Q, k, cap, tau, policy, batch, **kw):
    gpu = run_gpu(X.to(DEV), Q.to(DEV), k, cap, tau, policy, batch, **kw)
    return compare(X.numpy(), Q.numpy(), k, cap, tau, policy, gpu, rho=kw.get("rho", 1),
                   lsh_planes=kw.get("lsh_planes"), lsh_bucket=kw.get("lsh_bucket", 0), metric=kw.get("metric", "l2")), gpu


# ------------------------------------------------------------------ hand-traced sequences
@pytest.mark.parametrize("tr", all_traces(), ids=lambda t: t["name"])
@pytest.mark.parametrize("batch", [1, 3, 64])
def test_golden_traces_on_gpu(tr, batch):
    X, Q = torch.from_numpy(tr["corpus"]), torch.from_numpy(tr["queries"])
    ids, dists, hit, stats = run_gpu(X.to(DEV), Q.to(DEV), tr["k"], tr["capacity"], tr["tau"], tr["policy"], batch)
    assert np.array_equal(hit, tr["hit"])
    assert np.array_equal(ids, tr["ids"])
    assert stats["evictions"] == int((tr["evicted"] >= 0).sum())


def test_golden_trace_slots_via_probe():
    for tr in all_traces():
        X = torch.from_numpy(tr["corpus"]).to(DEV)
        p = prox.Prox(X, tr["k"], tr["capacity"], tr["tau"], tr["policy"])
        hit, slot, dist = p.probe_batch(torch.from_numpy(tr["queries"]).to(DEV))
        torch.cuda.synchronize()
        assert np.array_equal(hit.cpu().numpy(), tr["hit"]) and np.array_equal(slot.cpu().numpy(), tr["slot"])
        p.close()


@pytest.mark.parametrize("tr", all_load_traces(), ids=lambda t: t["name"])
@pytest.mark.parametrize("batch", [1, 4, 64])
def test_golden_traces_from_a_loaded_cache_on_gpu(tr, batch):
    """A bulk-loaded cache: which slot leaves first afterwards (hand-traced fixtures)."""
    X, Q = torch.from_numpy(tr["corpus"]).to(DEV), torch.from_numpy(tr["queries"]).to(DEV)
    for probe_only in (False, True):
        p = prox.Prox(X, tr["k"], tr["capacity"], tr["tau"], tr["policy"])
        p.cache_load(torch.from_numpy(tr["preload"]).to(DEV))
        hits, slots, ids = [], [], []
        for a in range(0, Q.shape[0], batch):
            if probe_only:
                h, s_, _ = p.probe_batch(Q[a:a + batch])
                slots.append(s_.clone())
            else:
                i_, _, h = p.query_batch(Q[a:a + batch])
                ids.append(i_.clone())
            hits.append(h.clone())
        torch.cuda.synchronize()
        assert p.status() == prox.OK
        st = p.stats()
        p.close()
        assert np.array_equal(torch.cat(hits).cpu().numpy(), tr["hit"])
        assert st["evictions"] == int((tr["evicted"] >= 0).sum())
        if probe_only:
            assert np.array_equal(torch.cat(slots).cpu().numpy(), tr["slot"])
        else:
            assert np.array_equal(torch.cat(ids).cpu().numpy(), tr["ids"])


# ------------------------------------------------------------------ the small sequential configuration
def test_tiny_sequential_config():
    c = W.CONFIGS["tiny"]
    X, Q, _, _ = W.build_workload(c, seed=0)
    res, _ = check(X, Q, c.k, c.capacity, c.taus[0], c.policy, c.batch)
    assert 0.0 < res["hit_rate"] < 1.0


# ------------------------------------------------------------------ batching must be unobservable
@pytest.mark.parametrize("policy", ["lru", "fifo"])
def test_batch_size_is_unobservable(policy):
    X, Q = stream(5003, 128, 16, 700, 60, 1.1, 0.02, seed=3)
    outs = []
    for batch in [1, 7, 64, 256, 1024]:
        res, gpu = check(X, Q, 10, 50, 0.5, policy, batch)
        outs.append(gpu)
    for g in outs[1:]:
        assert np.array_equal(g[0], outs[0][0]) and np.array_equal(g[2], outs[0][2])
        assert np.array_equal(g[1], outs[0][1])
    assert 0.05 < res["hit_rate"] < 0.99


# ------------------------------------------------------------------ tau sweep on a cut-down 1M-style stream
@pytest.mark.parametrize("tau", [0.0, 0.25, 0.5, 1.0, 2.0])
def test_tau_sweep_lru_batch64(tau):
    X, Q = stream(20011, 768, 32, 2500, 300, 1.1, 0.02, seed=1)
    res, gpu = check(X, Q, 10, 100, tau, "lru", 64)
    if tau == 0.0:
        assert res["hit_rate"] == 0.0
        ids, dists = oracle.exact_topk(X.numpy(), Q.numpy()[:50], 10)
        assert np.array_equal(gpu[0][:50], ids)              # tau = 0: plain kNN
    if tau == 2.0:
        assert res["hit_rate"] > 0.9


def test_k32_batch256_lru():
    X, Q = stream(30001, 768, 24, 1500, 200, 1.0, 0.03, seed=2)
    res, _ = check(X, Q, 32, 300, 1.0, "lru", 256)
    assert 0.0 < res["hit_rate"] < 1.0


def test_d128_batch1024_fifo_ragged_tail():
    X, Q = stream(50007, 128, 64, 2500, 700, 0.6, 0.05, seed=4)
    check(X, Q, 10, 500, 0.3, "fifo", 1024)


@pytest.mark.parametrize("metric,policy,batch", [("l2", "lru", 1), ("l2", "fifo", 4), ("cosine", "lru", 3), ("ip", "fifo", 2)])
def test_small_batches_over_a_small_corpus_take_the_short_route(metric, policy, batch):
    """Up to four queries per call, a cache of a few hundred keys and a corpus of a few thousand rows:
    the lookup is two launches and the database call one (every row measured in fp64); duplicate
    rows, hits on keys of the same call and evictions all occur."""
    X, Q = stream(6007, 256, 16, 700, 60, 1.0, 0.03, seed=81)
    X = X.clone()
    X[4000:4040] = X[100:140]                                          # equal rows: ties go to the lower id
    tau = {"l2": 0.4, "cosine": 0.2, "ip": -0.8}[metric]
    res, gpu = check(X, Q, 12, 25, tau, policy, batch, metric=metric)
    assert 0.2 < res["hit_rate"] < 0.97 and gpu[3]["evictions"] > 0
    if batch > 1:
        assert gpu[3]["intra_batch_hits"] > 0
    assert gpu[3]["uncertified"] == 0 and gpu[3]["scan_batches"] > 0


# ------------------------------------------------------------------ degenerate cases
def test_exact_duplicates_hit_at_tau_zero_in_and_across_batches():
    X, Q = stream(3000, 64, 8, 200, 200, 0.0, 0.05, seed=5)
    Q = Q.clone()
    Q[10] = Q[3]            # same batch (B = 64)
    Q[130] = Q[100]         # across batches
    Q[131] = Q[100]
    res, gpu = check(X, Q, 5, 150, 0.0, "lru", 64)
    hit = gpu[2]
    assert hit.sum() == 3 and hit[10] == 1 and hit[130] == 1 and hit[131] == 1
    assert np.array_equal(gpu[0][10], gpu[0][3]) and np.array_equal(gpu[0][131], gpu[0][100])


def test_huge_tau_everything_hits_the_first_key():
    X, Q = stream(2000, 64, 8, 300, 50, 1.0, 0.05, seed=6)
    res, gpu = check(X, Q, 8, 20, 4.5, "fifo", 128)
    assert gpu[2][0] == 0 and gpu[2][1:].all() and (gpu[0] == gpu[0][0]).all()
    assert gpu[3]["count"] == 1


@pytest.mark.parametrize("policy", ["lru", "fifo"])
@pytest.mark.parametrize("cap", [1, 5])
def test_capacity_smaller_than_batch(policy, cap):
    X, Q = stream(4000, 64, 8, 600, 40, 1.1, 0.03, seed=7)
    res, gpu = check(X, Q, 4, cap, 0.35, policy, 64)
    assert gpu[3]["evictions"] > 64 and 0.0 < res["hit_rate"] < 1.0


def test_corpus_smaller_than_candidate_count():
    for N, k in [(10, 10), (37, 5), (64, 64), (129, 3)]:
        X, Q = stream(N, 16, 2, 40, 10, 1.0, 0.05, seed=N)
        check(X, Q, k, 8, 0.01, "lru", 16)
        check(X, Q, k, 8, 0.01, "lru", 3)                    # the one-launch route of small batches


def test_uncertified_queries_take_the_exact_pass():
    # rows packed so tightly around one point that the bf16 scores cannot separate them
    g = torch.Generator().manual_seed(11)
    c = torch.randn(256, generator=g)
    X = c + 2e-4 * torch.randn(6000, 256, generator=g)
    X = X / X.norm(dim=1, keepdim=True)
    Q = X[:40] + 1e-4 * torch.randn(40, 256, generator=g)
    Q = (Q / Q.norm(dim=1, keepdim=True)).contiguous()
    X = X.contiguous()
    gpu = run_gpu(X.to(DEV), Q.to(DEV), 10, 16, 0.0, "lru", 8)
    assert gpu[3]["uncertified"] > 0 and gpu[3]["unresolved"] == 0
    ids, dists = oracle.exact_topk(X.numpy(), Q.numpy(), 10)
    assert np.array_equal(gpu[0], ids)
    assert np.allclose(gpu[1], dists, rtol=1e-4, atol=1e-12)


@pytest.mark.parametrize("metric", ["l2", "ip"])
def test_thousands_of_copies_of_one_row_are_still_answered_exactly(metric):
    """More rows tie at the k-th distance than the exact pass can collect (3000 copies of the row
    nearest to the query, scattered over the corpus): the answer is still the oracle's, the copies
    in id order, through the streaming pass that keeps every row it sees or proves it out."""
    g = torch.Generator().manual_seed(71)
    X = W.make_corpus(20000, 128, 16, seed=71)
    Q, _, _ = W.make_query_stream(X, 12, 3, 1.0, 0.02, seed=71)
    where = torch.randperm(20000, generator=g)[:3000]
    X = X.clone()
    X[where] = X[int(where[0])].clone()                               # 3000 identical rows
    Q = Q.clone()
    Q[:6] = (X[int(where[0])] + 0.01 * torch.randn(6, 128, generator=g))    # queries next to the copies
    Q = (Q / Q.norm(dim=1, keepdim=True)).contiguous()
    k = 10
    tau = 0.0 if metric == "l2" else -2.0
    gpu = run_gpu(X.to(DEV), Q.to(DEV), k, 16, tau, "lru", 6, metric=metric)       # (batches above four: the tensor-core route)
    ids, dists = oracle.exact_topk(X.numpy(), Q.numpy(), k, metric=parity.ORACLE_METRIC[metric])
    assert gpu[3]["unresolved"] == 0 and gpu[3]["hits"] == 0
    assert np.array_equal(gpu[0], ids)
    assert np.allclose(gpu[1], dists, rtol=1e-4, atol=1e-12)
    first_copies = np.sort(where.numpy())[:k]
    assert np.array_equal(gpu[0][0], first_copies)                     # ties come back in id order
    assert gpu[3]["uncertified"] >= 6


# ------------------------------------------------------------------ re-ranking factor (Section 3.3)
@pytest.mark.parametrize("policy,batch,rho,k", [("lru", 64, 4, 10), ("fifo", 1, 2, 5), ("lru", 200, 2, 32),
                                                ("fifo", 1024, 4, 32)])
def test_reranking_factor_matches_the_oracle(policy, batch, rho, k):
    """rho * k rows fetched and stored per miss, hits re-ranked against the current query: hits on
    stored keys, hits on keys of the same batch and capacity below the batch size all occur."""
    X, Q = stream(30011, 128, 48, 2300, 120, 1.0, 0.03, seed=31)
    res, gpu = check(X, Q, k, 40, 0.25, policy, batch, rho=rho)
    assert 0.3 < res["hit_rate"] < 0.97
    if batch > 1:
        assert gpu[3]["intra_batch_hits"] > 0
    # a re-ranked list differs from the stored head for a good share of the hits
    plain = run_gpu(X.to(DEV), Q.to(DEV), k, 40, 0.25, policy, batch, rho=1)
    h = res["ref"]["hit"] == 1
    assert (plain[0][h] != gpu[0][h]).any(axis=1).mean() > 0.05


def test_reranking_factor_argument_checks():
    Xd = torch.randn(500, 64, device=DEV).contiguous()
    lib = prox.load_library()
    for k, rho in [(10, 0), (33, 4), (64, 3), (10, 60)]:
        assert not lib.prox_create_rho(Xd.data_ptr(), 500, 64, k, 8, 0.5, 0, rho), (k, rho)
        assert "rho" in prox.last_error()
    h = lib.prox_create_rho(Xd.data_ptr(), 500, 64, 32, 8, 0.5, 0, 4)
    assert h
    lib.prox_destroy(h)


# ------------------------------------------------------------------ cosine distance (Section 2.2)
@pytest.mark.parametrize("policy,batch,rho", [("lru", 64, 1), ("fifo", 1, 1), ("lru", 500, 2)])
def test_cosine_distance_matches_the_oracle(policy, batch, rho):
    """Rows and queries of very different lengths: the Euclidean neighbours are not the cosine ones."""
    X, Q = stream(30011, 128, 48, 1500, 100, 1.0, 0.03, seed=51)
    g = torch.Generator().manual_seed(52)
    X = (X * (0.2 + 5.0 * torch.rand(X.shape[0], 1, generator=g))).contiguous()
    Q = (Q * (0.5 + 3.0 * torch.rand(Q.shape[0], 1, generator=g))).contiguous()
    res, gpu = check(X, Q, 10, 40, 0.12, policy, batch, rho=rho, metric="cosine")
    assert 0.2 < res["hit_rate"] < 0.97
    l2 = run_gpu(X.to(DEV), Q.to(DEV), 10, 40, 0.12, policy, batch, rho=rho)
    miss = res["ref"]["hit"] == 0
    assert (l2[0][miss] != gpu[0][miss]).any(axis=1).mean() > 0.5


def test_cosine_probe_only_with_loaded_keys():
    keys, centres = W.make_probe_keys(3000, 128, 256, seed=53)
    keys = (keys * (0.3 + 4.0 * torch.rand(3000, 1, generator=torch.Generator().manual_seed(54)))).contiguous()
    p = prox.Prox(keys[:64].contiguous().to(DEV), 1, 3000, 0.02, "lru", metric="cosine")
    p.cache_load(keys.to(DEV))
    o = oracle.Oracle(None, 128, 1, 3000, float(np.float32(0.02)), oracle.LRU, metric=oracle.COSINE)
    o.cache_load(keys.numpy())
    for b in range(2):
        Q = W.make_probe_batch(keys / keys.norm(dim=1, keepdim=True), centres, 512, 0.015, 53, b) * 2.5
        hit, slot, dist = p.probe_batch(Q.contiguous().to(DEV))
        torch.cuda.synchronize()
        r = o.query(Q.numpy())
        assert np.array_equal(hit.cpu().numpy(), r["hit"]) and np.array_equal(slot.cpu().numpy(), r["slot"])
        h = r["hit"] == 1
        assert np.allclose(dist.cpu().numpy()[h], r["best"][h], rtol=1e-4, atol=1e-9)
        assert 0.2 < r["hit"].mean() < 0.97
    assert p.status() == prox.OK
    p.close()


# ------------------------------------------------------------------ inner product (Section 2.2)
@pytest.mark.parametrize("policy,batch,rho,d,tau", [("lru", 64, 1, 128, -0.9), ("fifo", 1, 1, 128, -0.9), ("lru", 500, 2, 128, -0.9),
                                                    ("fifo", 256, 1, 768, -0.55), ("lru", 100, 1, 80, -0.9)])
def test_inner_product_matches_the_oracle(policy, batch, rho, d, tau):
    """Rows of very different lengths, so that the rows with the largest inner products are not the
    Euclidean neighbours; the tolerance is negative (a key matches when q.key >= 0.9 or 0.55).
    d = 80 is not a multiple of 64: that handle scans on the CUDA cores."""
    X, Q = stream(30011, d, 48, 1500, 100, 1.0, 0.03, seed=61)
    g = torch.Generator().manual_seed(62)
    X = (X * (0.5 + 1.5 * torch.rand(X.shape[0], 1, generator=g))).contiguous()
    res, gpu = check(X, Q, 10, 40, tau, policy, batch, rho=rho, metric="ip")
    assert 0.2 < res["hit_rate"] < 0.97
    assert (gpu[1] < 0).all()                                           # -(q.x) of the most similar rows
    l2 = run_gpu(X.to(DEV), Q.to(DEV), 10, 40, 0.3, policy, batch, rho=rho)
    miss = res["ref"]["hit"] == 0
    assert (l2[0][miss] != gpu[0][miss]).any(axis=1).mean() > 0.5


def test_inner_product_uncertified_queries_take_the_exact_pass():
    """Rows packed so tightly that the bf16 products cannot separate them: both sweeps of the
    exact pass run with the inner product's margins."""
    g = torch.Generator().manual_seed(63)
    c = torch.randn(256, generator=g)
    X = c + 2e-4 * torch.randn(6000, 256, generator=g)
    X = (X / X.norm(dim=1, keepdim=True)).contiguous()
    Q = X[:40] + 1e-4 * torch.randn(40, 256, generator=g)
    Q = (Q / Q.norm(dim=1, keepdim=True)).contiguous()
    gpu = run_gpu(X.to(DEV), Q.to(DEV), 10, 16, -2.0, "lru", 8, metric="ip")          # -q.x <= -2 never holds: all miss
    assert gpu[3]["uncertified"] > 0 and gpu[3]["unresolved"] == 0 and gpu[3]["hits"] == 0
    ids, dists = oracle.exact_topk(X.numpy(), Q.numpy(), 10, metric=oracle.IP)
    assert np.array_equal(gpu[0], ids)
    assert np.allclose(gpu[1], dists, rtol=1e-4, atol=1e-12)


def test_inner_product_probe_only_and_argument_checks():
    keys, centres = W.make_probe_keys(3000, 128, 256, seed=64)
    keys = (keys * (0.5 + 1.5 * torch.rand(3000, 1, generator=torch.Generator().manual_seed(65)))).contiguous()
    tau = -1.7                                                          # only the longer keys of a component match
    p = prox.Prox(keys[:64].contiguous().to(DEV), 1, 3000, tau, "lru", metric="ip")
    p.cache_load(keys.to(DEV))
    o = oracle.Oracle(None, 128, 1, 3000, float(np.float32(tau)), oracle.LRU, metric=oracle.IP)
    o.cache_load(keys.numpy())
    for b in range(2):
        Q = W.make_probe_batch(keys / keys.norm(dim=1, keepdim=True), centres, 512, 0.015, 64, b)
        hit, slot, dist = p.probe_batch(Q.contiguous().to(DEV))
        torch.cuda.synchronize()
        r = o.query(Q.numpy())
        assert np.array_equal(hit.cpu().numpy(), r["hit"]) and np.array_equal(slot.cpu().numpy(), r["slot"])
        h = r["hit"] == 1
        assert np.allclose(dist.cpu().numpy()[h], r["best"][h], rtol=1e-6)
        assert 0.1 < r["hit"].mean() < 0.97
    assert p.status() == prox.OK
    p.close()
    lib = prox.load_library()
    Xd = keys.to(DEV)
    assert not lib.prox_create_metric(Xd.data_ptr(), 3000, 128, 4, 8, -0.5, 0, 1, prox.METRIC_L2SQ)       # negative tau: inner product only
    assert not lib.prox_create_metric(Xd.data_ptr(), 3000, 128, 4, 8, -0.5, 0, 1, prox.METRIC_COSINE)
    assert not lib.prox_create_metric(Xd.data_ptr(), 3000, 128, 4, 8, float("nan"), 0, 1, prox.METRIC_IP)
    assert not lib.prox_create_metric(Xd.data_ptr(), 3000, 128, 4, 8, 0.5, 0, 1, 3)
    h = lib.prox_create_metric(Xd.data_ptr(), 3000, 128, 4, 8, -0.5, 0, 1, prox.METRIC_IP)
    assert h
    lib.prox_destroy(h)


# ------------------------------------------------------------------ PROXIMITY-LSH (Section 3.2)
@pytest.mark.parametrize("policy,batch,L,b,rho", [("lru", 1, 4, 3, 1), ("fifo", 64, 4, 3, 1), ("lru", 1000, 6, 2, 1),
                                                  ("fifo", 256, 0, 7, 1), ("lru", 300, 5, 4, 2)])
def test_lsh_cache_matches_the_oracle(policy, batch, L, b, rho):
    """Buckets of a few entries and batches far larger than a bucket: hits on stored keys, on keys
    of the same batch, and evictions of entries that the same batch inserted all occur."""
    X, Q = stream(20011, 128, 32, 2400, 150, 0.9, 0.03, seed=41)
    planes = torch.randn(L, 128, generator=torch.Generator().manual_seed(5)).numpy()
    res, gpu = check(X, Q, 8, (1 << L) * b, 0.3, policy, batch, rho=rho, lsh_planes=planes, lsh_bucket=b)
    assert 0.1 < res["hit_rate"] < 0.97
    assert gpu[3]["evictions"] == int((res["ref"]["evicted"] >= 0).sum()) > 0
    if batch > 1:
        assert gpu[3]["intra_batch_hits"] > 0


def test_lsh_probe_only_slots_and_argument_checks():
    X, Q = stream(5000, 64, 16, 700, 60, 0.9, 0.03, seed=42)
    planes = torch.randn(5, 64, generator=torch.Generator().manual_seed(6))
    p = prox.Prox(X.to(DEV), 4, 32 * 3, 0.3, "lru", lsh_planes=planes.to(DEV), lsh_bucket=3)
    o = oracle.Oracle(None, 64, 4, 32 * 3, float(np.float32(0.3)), oracle.LRU, lsh_planes=planes.numpy(), lsh_bucket=3)
    for a in range(0, 700, 350):
        hit, slot, dist = p.probe_batch(Q[a:a + 350].to(DEV))
        torch.cuda.synchronize()
        r = o.query(Q[a:a + 350].numpy())
        assert np.array_equal(hit.cpu().numpy(), r["hit"]) and np.array_equal(slot.cpu().numpy(), r["slot"])
    assert p.status() == prox.OK
    with pytest.raises(prox.ProxError):
        p.cache_load(Q[:8].to(DEV))
    p.close()
    lib = prox.load_library()
    Xd = X.to(DEV)
    for L, b in [(-1, 4), (21, 4), (3, 0), (3, 65)]:
        assert not lib.prox_create_lsh(Xd.data_ptr(), 5000, 64, 4, L, b, planes.to(DEV).data_ptr(), 0.3, 0, 1)


# ------------------------------------------------------------------ probe only, pre-filled cache
@pytest.mark.parametrize("policy", ["lru", "fifo"])
@pytest.mark.parametrize("n_keys", [3000, 6000])        # fp64 probe / coarse tensor-core probe with exact recheck
def test_probe_only_prefilled_cache(policy, n_keys):
    keys, centres = W.make_probe_keys(n_keys, 768, 4096, seed=8)
    p = prox.Prox(keys[:64].contiguous().to(DEV), 1, n_keys, 0.5, policy)
    p.cache_load(keys.to(DEV))
    o = oracle.Oracle(None, 768, 1, n_keys, float(np.float32(0.5)), oracle.LRU if policy == "lru" else oracle.FIFO)
    o.cache_load(keys.numpy())
    for b in range(3):
        Q = W.make_probe_batch(keys, centres, 1024, 0.02, 8, b)
        hit, slot, dist = p.probe_batch(Q.to(DEV))
        torch.cuda.synchronize()
        r = o.query(Q.numpy())
        assert np.array_equal(hit.cpu().numpy(), r["hit"])
        assert np.array_equal(slot.cpu().numpy(), r["slot"])
        h = r["hit"] == 1
        assert np.allclose(dist.cpu().numpy()[h], r["best"][h], rtol=1e-6)
        assert 0.3 < r["hit"].mean() < 0.97
    assert p.status() == prox.OK
    p.close()


@pytest.mark.parametrize("policy", ["lru", "fifo"])
@pytest.mark.parametrize("n_keys,batch,d", [(1024, 1024, 768), (1024, 1000, 64), (2048, 1024, 64), (700, 1024, 64), (300, 512, 64)])
@pytest.mark.parametrize("in_order", [False, True])
def test_probe_only_cache_as_small_as_the_batch(policy, n_keys, batch, d, in_order):
    """A full cache of about as many keys as the batch has queries: every key is at risk, every hit
    is on a key that an earlier miss of the same batch may have evicted, and a third of the batch
    is near an earlier query of the batch.  The replay solves such a batch as a fixed point; with
    the cross-check mode it runs in query order.  Both against the oracle, flag by flag and slot
    by slot, over several batches (the state carries over).  Capacities below the batch size use
    up the at-risk list, which the fixed-point replay leaves to the in-order one."""
    keys, centres = W.make_probe_keys(n_keys, d, 4 * n_keys, seed=31)      # most fresh draws find no key of their component
    tau = 0.5 if d == 768 else 0.02
    p = prox.Prox(keys[:64].contiguous().to(DEV), 1, n_keys, tau, policy)
    if in_order:
        p.set_scan_mode(prox.SCAN_CUDA_CORE)
    p.cache_load(keys.to(DEV))
    o = oracle.Oracle(None, d, 1, n_keys, float(np.float32(tau)), oracle.LRU if policy == "lru" else oracle.FIFO)
    o.cache_load(keys.numpy())
    gen = torch.Generator().manual_seed(77)
    rates = []
    for b in range(4):
        Q = W.make_probe_batch(keys, centres, batch, 0.02 if d == 768 else 0.01, 31, b)
        # a third of the queries repeat, slightly moved, an earlier query of the same batch
        idx = torch.randperm(batch, generator=gen)[: batch // 3]
        src = (torch.rand(batch // 3, generator=gen) * idx.float()).long()
        moved = Q[src] + 1e-3 * torch.randn(batch // 3, d, generator=gen)
        Q[idx] = torch.where((idx > 0)[:, None], moved, Q[idx])
        hit, slot, dist = p.probe_batch(Q.to(DEV))
        torch.cuda.synchronize()
        r = o.query(Q.numpy())
        assert np.array_equal(hit.cpu().numpy(), r["hit"]), f"batch {b}: first differing flag at {np.nonzero(hit.cpu().numpy() != r['hit'])[0][:1]}"
        assert np.array_equal(slot.cpu().numpy(), r["slot"]), f"batch {b}: first differing slot at {np.nonzero(slot.cpu().numpy() != r['slot'])[0][:1]}"
        h = r["hit"] == 1
        assert np.allclose(dist.cpu().numpy()[h], r["best"][h], rtol=1e-6)
        rates.append(float(r["hit"].mean()))
    assert 0.05 < np.mean(rates) < 0.98, rates
    assert p.status() == prox.OK
    st = p.stats()
    p.close()
    if in_order:
        assert st["parallel_replays"] == 0
    elif n_keys >= batch:
        assert st["parallel_replays"] >= 3, st
    assert st["intra_batch_hits"] > 0


@pytest.mark.parametrize("policy", ["lru", "fifo"])
def test_probe_only_cache_above_the_multi_block_risk_selection(policy):
    """More than 65536 keys: the at-risk entries are picked by the histogram kernels spread over
    the GPU; the slots that misses overwrite show the eviction order."""
    n_keys, d = 70000, 64
    keys, centres = W.make_probe_keys(n_keys, d, 512, seed=21)
    tau = 0.02                                              # queries around keys hit, fresh draws mostly miss
    p = prox.Prox(keys[:64].contiguous().to(DEV), 1, n_keys, tau, policy)
    p.cache_load(keys.to(DEV))
    o = oracle.Oracle(None, d, 1, n_keys, float(np.float32(tau)), oracle.LRU if policy == "lru" else oracle.FIFO)
    o.cache_load(keys.numpy())
    misses = 0
    for b in range(4):
        Q = W.make_probe_batch(keys, centres, 1000, 0.01, 21, b)
        hit, slot, dist = p.probe_batch(Q.to(DEV))
        torch.cuda.synchronize()
        r = o.query(Q.numpy())
        assert np.array_equal(hit.cpu().numpy(), r["hit"])
        assert np.array_equal(slot.cpu().numpy(), r["slot"])
        misses += int((r["hit"] == 0).sum())
    assert 100 < misses < 3900
    assert p.status() == prox.OK
    p.close()


@pytest.mark.parametrize("n_keys,n_batches,batch,policies", [(1 << 17, 2, 1024, ("lru", "fifo")), (1 << 20, 1, 256, ("lru",))])
def test_probe_only_at_the_benchmarked_cache_sizes(n_keys, n_batches, batch, policies):
    """The probe-only workload at the sizes the benchmark reports (2^17 and 2^20 keys of 768
    dimensions, full cache, tau = 0.5): every flag, matched or written slot and hit distance against
    the oracle.  The oracle walks all keys for every query on one core (a minute or two per batch),
    so its runs go to worker processes and overlap the GPU side and one another; the cache state is
    sequential, so a batch cannot be sampled: at 2^20 keys one batch of 256 queries is replayed."""
    d, tau = 768, 0.5
    # two keys per mixture component on average: about one fresh draw in seven finds no key of its
    # component in the cache and misses, so every batch also evicts and inserts
    keys, centres = W.make_probe_keys(n_keys, d, n_keys // 2, seed=8)
    Qs = torch.stack([W.make_probe_batch(keys, centres, batch, 0.02, 8, b) for b in range(n_batches)])
    kb, kdesc = oracle_workers.share(keys.numpy())
    qb, qdesc = oracle_workers.share(Qs.numpy())
    try:
        with oracle_workers.pool(len(policies)) as pool:
            jobs = [pool.apply_async(oracle_workers.probe_trace_worker, (kdesc, qdesc, tau, pol)) for pol in policies]
            keys_d, got = keys.to(DEV), {}
            for pol in policies:
                p = prox.Prox(keys_d[:64].contiguous(), 1, n_keys, tau, pol)
                p.cache_load(keys_d)
                got[pol] = []
                for b in range(n_batches):
                    hit, slot, dist = p.probe_batch(Qs[b].to(DEV))
                    got[pol].append((hit.cpu().numpy(), slot.cpu().numpy(), dist.cpu().numpy()))
                torch.cuda.synchronize()
                assert p.status() == prox.OK, prox.last_error()
                got[pol].append(p.stats())
                p.close()
            for pol, job in zip(policies, jobs):
                ref = job.get(timeout=900)
                evictions = 0
                for b in range(n_batches):
                    hit, slot, dist = got[pol][b]
                    r = ref[b]
                    assert np.array_equal(hit, r["hit"]), f"{pol} batch {b}: first differing flag at {np.nonzero(hit != r['hit'])[0][:1]}"
                    assert np.array_equal(slot, r["slot"]), f"{pol} batch {b}: first differing slot at {np.nonzero(slot != r['slot'])[0][:1]}"
                    h = r["hit"] == 1
                    assert np.allclose(dist[h], r["best"][h], rtol=1e-6)
                    assert 0.3 < r["hit"].mean() < 0.99
                    evictions += int((r["evicted"] >= 0).sum())
                assert got[pol][n_batches]["evictions"] == evictions > 0
    finally:
        for blk in (kb, qb):
            blk.close()
            blk.unlink()


def test_large_cache_stream_with_coarse_probe():
    """Capacity above the switch-over to the tensor-core probe, pre-filled and full, so that the
    stream evicts from its first miss on; lists of pre-filled keys are the empty ones on both sides."""
    X, Q = stream(20011, 256, 64, 1600, 3000, 0.8, 0.03, seed=13)
    keys = torch.cat([Q[800:], W.make_corpus(4400, 256, 64, seed=14)]).contiguous()     # some keys near later queries
    Qs = Q[:800].contiguous()
    k, cap, tau = 10, keys.shape[0], 0.5
    p = prox.Prox(X.to(DEV), k, cap, tau, "lru")
    p.cache_load(keys.to(DEV))
    outs = [p.query_batch(Qs[a:a + 800].to(DEV)) for a in range(0, 800, 800)]      # 800 x 5200 pairs: coarse probe
    torch.cuda.synchronize()
    assert p.status() == prox.OK
    st = p.stats()
    p.close()
    ids = torch.cat([o_[0] for o_ in outs]).cpu().numpy()
    dists = torch.cat([o_[1] for o_ in outs]).cpu().numpy()
    hit = torch.cat([o_[2] for o_ in outs]).cpu().numpy()
    o = oracle.Oracle(X.numpy(), 256, k, cap, float(np.float32(tau)), oracle.LRU)
    o.cache_load(keys.numpy())
    r = o.query(Qs.numpy())
    assert np.array_equal(hit, r["hit"]) and 0.05 < r["hit"].mean() < 0.97
    assert np.array_equal(ids, r["ids"])
    assert np.allclose(dists, r["dists"], rtol=1e-4, atol=1e-12)
    assert st["evictions"] == int((r["evicted"] >= 0).sum()) > 0


def test_coarse_probe_hands_tight_clusters_to_the_exact_probe():
    g = torch.Generator().manual_seed(17)
    c = torch.randn(128, generator=g)
    keys = c + 3e-4 * torch.randn(5000, 128, generator=g)
    keys = (keys / keys.norm(dim=1, keepdim=True)).contiguous()
    Q = keys[:700] + 1e-4 * torch.randn(700, 128, generator=g)       # 700 x 5000 pairs: above the switch to the coarse probe
    Q = (Q / Q.norm(dim=1, keepdim=True)).contiguous()
    tau = 1.22e-6
    p = prox.Prox(keys[:64].contiguous().to(DEV), 1, 5000, tau, "fifo")
    p.cache_load(keys.to(DEV))
    hit, slot, dist = p.probe_batch(Q.to(DEV))
    torch.cuda.synchronize()
    st = p.stats()
    assert p.status() == prox.OK
    p.close()
    o = oracle.Oracle(None, 128, 1, 5000, float(np.float32(tau)), oracle.FIFO)
    o.cache_load(keys.numpy())
    r = o.query(Q.numpy())
    assert st["probe_uncertified"] > 0
    assert np.array_equal(hit.cpu().numpy(), r["hit"]) and np.array_equal(slot.cpu().numpy(), r["slot"])
    assert 0.05 < r["hit"].mean() < 0.999


# ------------------------------------------------------------------ API behaviour
def test_host_buffer_entry_point_equals_device_entry_point():
    X, Q = stream(6001, 128, 8, 300, 40, 1.1, 0.02, seed=9)
    a = run_gpu(X.to(DEV), Q.to(DEV), 10, 30, 0.5, "lru", 64)
    b = run_gpu(X.to(DEV), Q.to(DEV), 10, 30, 0.5, "lru", 64, host_api=True)
    for x, y in zip(a[:3], b[:3]):
        assert np.array_equal(x, y)


@pytest.mark.parametrize("policy,batch,d,kw", [("fifo", 1, 768, {}), ("lru", 64, 128, {}), ("lru", 3, 64, {"rho": 2}),
                                               ("fifo", 200, 128, {"metric": "cosine"}), ("lru", 1, 128, {"metric": "ip"})])
def test_recorded_batches_replay_the_plain_call(policy, batch, d, kw):
    """prox_record_batch / prox_replay_batch: the batch call captured once on fixed buffers and
    replayed for a stream of batches, against the oracle (the cache state carries over from replay
    to replay) and, output for output and counter for counter, against the plain call."""
    X, Q = stream(9001, d, 16, 900 if batch > 1 else 300, 400, 0.8, 0.02, seed=23)
    l2 = {768: 0.7, 128: 0.13, 64: 0.08}[d]                    # about the squared distance of two noisy copies of a topic
    tau = {"ip": l2 / 2 - 1.0, "cosine": l2 / 2}.get(kw.get("metric"), l2)
    res, gpu = check(X, Q, 10, 50, tau, policy, batch, recorded=True, **kw)
    assert 0.0 < res["hit_rate"] < 1.0
    plain = run_gpu(X.to(DEV), Q.to(DEV), 10, 50, tau, policy, batch, **kw)
    for x, y in zip(gpu[:3], plain[:3]):
        assert np.array_equal(x, y)
    assert gpu[3] == plain[3]


def test_recording_argument_checks():
    X, Q = stream(3001, 64, 8, 64, 20, 1.1, 0.02, seed=24)
    p = prox.Prox(X.to(DEV), 5, 20, 0.5, "lru")
    q = Q[:8].to(DEV)
    ids = torch.empty(8, 5, dtype=torch.int64, device=DEV)
    dist = torch.empty(8, 5, dtype=torch.float32, device=DEV)
    hit = torch.empty(8, dtype=torch.uint8, device=DEV)
    side = torch.cuda.Stream()
    p.profile(None)
    with pytest.raises(prox.ProxError, match="prox_profile"):
        p.record_batch(q, ids, dist, hit, stream=side)
    p.profile(())
    with pytest.raises(prox.ProxError):
        p.record_batch(q, ids, dist, hit.to(torch.int32), stream=side)
    launches = p.kernel_launches()
    rec = p.record_batch(q, ids, dist, hit, stream=side)
    assert p.kernel_launches() == launches and p.stats()["queries"] == 0      # recording runs nothing
    rec.replay(stream=side)
    side.synchronize()
    assert p.stats()["queries"] == 8 and p.kernel_launches() > launches
    assert p.status() == prox.OK
    rec.close()
    rec.close()
    p.close()


@pytest.mark.parametrize("d,batch", [(768, 64), (128, 256), (256, 24), (128, 600), (128, 300), (64, 1000)])
def test_the_three_scan_kernels_agree(d, batch):
    """Two-block tensor-core scan (default), one-block tensor-core scan and CUDA-core scan."""
    X, Q = stream(9001, d, 8, 520, 40, 1.1, 0.02, seed=10)
    a = run_gpu(X.to(DEV), Q.to(DEV), 10, 30, 0.25, "lru", batch)
    b = run_gpu(X.to(DEV), Q.to(DEV), 10, 30, 0.25, "lru", batch, scan_mode=prox.SCAN_CUDA_CORE)
    c = run_gpu(X.to(DEV), Q.to(DEV), 10, 30, 0.25, "lru", batch, scan_mode=prox.SCAN_TC_SINGLE)
    for x, y, z in zip(a[:3], b[:3], c[:3]):
        assert np.array_equal(x, y) and np.array_equal(x, z)
    ids, dists = oracle.exact_topk(X.numpy(), Q.numpy()[:40], 10)
    miss = a[2][:40] == 0
    assert np.array_equal(a[0][:40][miss], ids[miss])


def test_reset_cache_and_argument_checks():
    X, Q = stream(2000, 64, 4, 128, 20, 1.0, 0.02, seed=12)
    Xd, Qd = X.to(DEV), Q.to(DEV)
    p = prox.Prox(Xd, 5, 32, 0.5, "lru")
    a = [t.clone() for t in p.query_batch(Qd)]
    p.reset_cache()
    b = p.query_batch(Qd)
    torch.cuda.synchronize()
    for x, y in zip(a, b):
        assert torch.equal(x, y)
    assert p.stats()["queries"] == 128
    lib = prox.load_library()
    assert lib.prox_query_batch(p._h, Qd.data_ptr(), 0, b[0].data_ptr(), b[1].data_ptr(), b[2].data_ptr(), None) == prox.ERR_INVALID_ARG
    assert lib.prox_query_batch(p._h, Qd.data_ptr(), 1025, b[0].data_ptr(), b[1].data_ptr(), b[2].data_ptr(), None) == prox.ERR_INVALID_ARG
    assert lib.prox_query_batch(p._h, None, 4, b[0].data_ptr(), b[1].data_ptr(), b[2].data_ptr(), None) == prox.ERR_INVALID_ARG
    p.close()
    for bad in [dict(k=0), dict(k=65), dict(capacity=0), dict(tau=-1.0), dict(tau=float("nan")), dict(policy=2)]:
        args = dict(k=5, capacity=8, tau=0.5, policy=0)
        args.update(bad)
        assert not lib.prox_create(Xd.data_ptr(), 2000, 64, args["k"], args["capacity"], args["tau"], args["policy"])
        assert prox.last_error() != ""
    assert not lib.prox_create(Xd.data_ptr(), 2000, 60, 5, 8, 0.5, 0)      # d not a multiple of 16
