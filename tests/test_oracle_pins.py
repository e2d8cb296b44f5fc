"""Pins of the CPU oracle against things other than itself: closed forms, an independent
numpy brute force, the invariants that Algorithm 1 and Section 3.3 of the paper imply,
hand-traced eviction sequences, and the paper's own operation count (Section 3.2)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05530_b200 import workloads as W
from golden_traces import all_load_traces, all_traces

POL = {"lru": oracle.LRU, "fifo": oracle.FIFO}


def unit_rows(n, d, seed):
    r = np.random.default_rng(seed).standard_normal((n, d))
    return (r / np.linalg.norm(r, axis=1, keepdims=True)).astype(np.float32)


# ---------------------------------------------------------------- distance (Algorithm 1, distance(q, k))
def test_sqdist_closed_forms():
    assert oracle.sqdist([1, 2, 3], [4, 6, 8]) == 50.0           # 9 + 16 + 25
    e = np.eye(8, dtype=np.float32)
    for i in range(8):
        for j in range(8):
            assert oracle.sqdist(e[i], e[j]) == (0.0 if i == j else 2.0)   # orthonormal basis
    a = unit_rows(5, 768, 0)
    for i in range(5):
        assert oracle.sqdist(a[i], a[i]) == 0.0                   # duplicates: exactly zero
        for j in range(5):                                        # |a-b|^2 = |a|^2 + |b|^2 - 2 a.b
            a64, b64 = a[i].astype(np.float64), a[j].astype(np.float64)
            closed = a64 @ a64 + b64 @ b64 - 2 * (a64 @ b64)
            assert abs(oracle.sqdist(a[i], a[j]) - closed) < 1e-12
            assert oracle.sqdist(a[i], a[j]) == oracle.sqdist(a[j], a[i])
    # not a dot product, not an unsquared norm, not a difference without the square
    assert oracle.sqdist([3, 0], [0, 4]) == 25.0
    assert oracle.sqdist([-1, -1], [1, 1]) == 8.0


# ---------------------------------------------------------------- database call (Algorithm 1, retrieveDocumentIndices)
@pytest.mark.parametrize("n,d,k,seed", [(50, 3, 5, 0), (1000, 16, 10, 1), (777, 128, 32, 2), (64, 768, 64, 3)])
def test_exact_topk_vs_numpy_bruteforce(n, d, k, seed):
    X = unit_rows(n, d, seed)
    Q = unit_rows(7, d, seed + 100)
    ids, dists = oracle.exact_topk(X, Q, k)
    X64, Q64 = X.astype(np.float64), Q.astype(np.float64)
    for i in range(Q.shape[0]):
        full = ((X64 - Q64[i]) ** 2).sum(1)
        order = np.lexsort((np.arange(n), full))[:k]              # by distance, then id
        assert np.array_equal(ids[i], order)
        assert np.allclose(dists[i], full[order], rtol=1e-13, atol=0)
        assert np.all(np.diff(dists[i]) >= 0)                     # "sorted list" (Section 3)


def test_exact_topk_planted_ties_and_permutation():
    X = unit_rows(300, 32, 5)
    q = unit_rows(1, 32, 6)[0]
    X[17] = q                                                     # planted exact neighbour
    X[250] = X[40]                                                # duplicate rows: equal distance
    ids, dists = oracle.exact_topk(X, q, 300)
    assert ids[0, 0] == 17 and dists[0, 0] == 0.0
    p40, p250 = np.where(ids[0] == 40)[0][0], np.where(ids[0] == 250)[0][0]
    assert p250 == p40 + 1                                        # tie: lower id first
    perm = np.random.default_rng(0).permutation(300)
    ids_p, dists_p = oracle.exact_topk(X[perm], q, 20)
    ids_s, dists_s = oracle.exact_topk(X, q, 20)
    assert np.array_equal(dists_p, dists_s)                       # same multiset of rows
    assert set(perm[ids_p[0]]) == set(ids_s[0])


def test_chunked_topk_equals_whole():
    X, q = unit_rows(1000, 24, 7), unit_rows(1, 24, 8)[0]
    X[900] = X[3]
    whole_ids, whole_d = oracle.exact_topk(X, q, 1000)
    ch = oracle.ChunkedTopK(q, 1000)
    for a, b in [(0, 1), (1, 333), (333, 334), (334, 1000)]:
        ch.feed(X[a:b])
    assert np.array_equal(ch.ids, whole_ids[0]) and np.array_equal(ch.dists, whole_d[0])


# ---------------------------------------------------------------- invariants of Algorithm 1
def small_workload(seed=0, N=400, d=32, nq=120, topics=15):
    torch.manual_seed(0)
    X = W.make_corpus(N, d, 8, seed)
    q, ranks, rows = W.make_query_stream(X, nq, topics, 1.1, 0.02, seed)
    return X.numpy(), q.numpy(), ranks.numpy()


@pytest.mark.parametrize("policy", ["lru", "fifo"])
def test_tau_zero_without_duplicates_is_plain_knn(policy):
    X, Q, _ = small_workload()
    o = oracle.Oracle(X, X.shape[1], 5, 10, 0.0, POL[policy])
    r = o.query(Q)
    assert r["hit"].sum() == 0                                    # tau = 0: exact matching only (Section 3.3.3)
    ids, dists = oracle.exact_topk(X, Q, 5)
    assert np.array_equal(r["ids"], ids) and np.array_equal(r["dists"], dists)
    c = o.counters()
    assert c["misses"] == len(Q) and c["evictions"] == len(Q) - 10 and c["count"] == 10


@pytest.mark.parametrize("tau", [0.0, 0.3])
def test_exact_duplicate_of_resident_key_hits(tau):
    X, Q, _ = small_workload(1)
    Q = Q.copy()
    Q[50] = Q[47]                                                 # 47 is still resident (capacity 10 > 3)
    o = oracle.Oracle(X, X.shape[1], 4, 10, tau, oracle.LRU)
    r = o.query(Q)
    if tau == 0.0:
        assert r["hit"].sum() == 1
    assert r["hit"][50] == 1
    assert np.array_equal(r["ids"][50], r["ids"][r["origin"][50]])
    if r["hit"][47] == 0:                                         # 47 became a key: its copy is at distance 0
        assert r["best"][50] == 0.0 and r["origin"][50] == 47
    else:                                                         # 47 hit a key that LRU kept: the copy sees the same
        assert r["best"][50] <= r["best"][47] and r["best"][50] <= tau


def test_huge_tau_every_later_query_hits_first_key():
    X, Q, _ = small_workload(2)
    o = oracle.Oracle(X, X.shape[1], 6, 10, 4.0 + 1e-6, oracle.FIFO)   # unit vectors: distance <= 4
    r = o.query(Q)
    assert r["hit"][0] == 0 and r["hit"][1:].all()
    assert (r["slot"] == 0).all() and (r["origin"] == 0).all()
    assert (r["ids"] == r["ids"][0]).all() and (r["dists"] == r["dists"][0]).all()
    assert o.counters()["count"] == 1 and o.counters()["evictions"] == 0
    ids0, _ = oracle.exact_topk(X, Q[0], 6)
    assert np.array_equal(r["ids"][0], ids0[0])


@pytest.mark.parametrize("policy", ["lru", "fifo"])
def test_capacity_one(policy):
    X, Q, _ = small_workload(3)
    tau = 0.2
    o = oracle.Oracle(X, X.shape[1], 3, 1, tau, POL[policy])
    r = o.query(Q)
    last_miss = -1
    for i in range(len(Q)):
        if last_miss >= 0:
            dist = float(((Q[i].astype(np.float64) - Q[last_miss].astype(np.float64)) ** 2).sum())
            assert r["hit"][i] == (dist <= tau)                   # only the most recent miss is resident
            assert abs(r["best"][i] - dist) < 1e-12
        else:
            assert r["hit"][i] == 0 and np.isinf(r["best"][i])     # empty cache: a miss
        if r["hit"][i]:
            assert r["origin"][i] == last_miss and np.array_equal(r["ids"][i], r["ids"][last_miss])
        else:
            assert r["slot"][i] == 0 and r["evicted"][i] == (0 if last_miss >= 0 else -1)
            last_miss = i
    assert 0 < r["hit"].sum() < len(Q)


def test_hit_returns_nearest_key_and_eviction_only_when_full():
    X, Q, _ = small_workload(4, nq=200)
    cap, tau = 12, 0.15
    o = oracle.Oracle(X, X.shape[1], 3, cap, tau, oracle.LRU)
    r = o.query(Q)
    # replay with an independent dict-based model written straight from Algorithm 1
    keys, stamp = {}, {}
    Q64 = Q.astype(np.float64)
    for i in range(len(Q)):
        dist = {s: float(((Q64[i] - Q64[j]) ** 2).sum()) for s, j in keys.items()}
        best = min(dist, key=lambda s: (dist[s], s)) if dist else None
        if best is not None and dist[best] <= tau:
            assert r["hit"][i] == 1 and r["slot"][i] == best and r["origin"][i] == keys[best]
            stamp[best] = i
        else:
            assert r["hit"][i] == 0
            if len(keys) >= cap:                                  # evict only when |C| >= c
                victim = min(stamp, key=stamp.get)
                assert r["evicted"][i] == victim
                del keys[victim], stamp[victim]
                slot = victim
            else:
                assert r["evicted"][i] == -1
                slot = len(keys)
            assert r["slot"][i] == slot
            keys[slot], stamp[slot] = i, i
    assert 0 < r["hit"].sum() < len(Q) and o.counters()["evictions"] > 0


def test_hit_rate_grows_with_tau_on_the_synthetic_stream():
    X, Q, _ = small_workload(5, nq=300)
    rates = []
    for tau in [0.0, 0.02, 0.1, 0.5, 2.0, 4.1]:
        o = oracle.Oracle(None, X.shape[1], 1, 20, tau, oracle.LRU)
        rates.append(o.query(Q)["hit"].mean())
    assert rates[0] == 0.0 and rates[-1] == (len(Q) - 1) / len(Q)
    assert all(b >= a for a, b in zip(rates, rates[1:]))


# ---------------------------------------------------------------- hand-traced eviction orders
@pytest.mark.parametrize("tr", all_traces(), ids=lambda t: t["name"])
def test_golden_traces(tr):
    o = oracle.Oracle(tr["corpus"], tr["corpus"].shape[1], tr["k"], tr["capacity"], tr["tau"], POL[tr["policy"]])
    r = o.query(tr["queries"])
    assert np.array_equal(r["hit"], tr["hit"])
    assert np.array_equal(r["slot"], tr["slot"])
    assert np.array_equal(r["evicted"], tr["evicted"])
    assert np.array_equal(r["ids"], tr["ids"])


@pytest.mark.parametrize("tr", all_load_traces(), ids=lambda t: t["name"])
def test_golden_traces_from_a_loaded_cache(tr):
    """Bulk load: which entry leaves first afterwards (hand-traced, Section 3.3.2)."""
    o = oracle.Oracle(tr["corpus"], tr["corpus"].shape[1], tr["k"], tr["capacity"], tr["tau"], POL[tr["policy"]])
    o.cache_load(tr["preload"])
    assert o.counters()["count"] == len(tr["preload"])
    r = o.query(tr["queries"])
    assert np.array_equal(r["hit"], tr["hit"])
    assert np.array_equal(r["slot"], tr["slot"])
    assert np.array_equal(r["evicted"], tr["evicted"])
    assert np.array_equal(r["ids"], tr["ids"])


@pytest.mark.parametrize("policy", ["lru", "fifo"])
def test_loaded_cache_equals_the_same_keys_inserted_by_misses(policy):
    """A bulk load of n distinct keys must leave the cache as n misses on those keys would (tau = 0:
    no hits): same slots, same eviction order afterwards, whatever the policy."""
    X, Q, _ = small_workload(8, nq=90)
    n, cap = 12, 12
    a = oracle.Oracle(None, X.shape[1], 1, cap, 0.05, POL[policy])
    a.cache_load(Q[:n])
    b = oracle.Oracle(None, X.shape[1], 1, cap, 0.0, POL[policy])
    rb0 = b.query(Q[:n])
    assert rb0["hit"].sum() == 0 and np.array_equal(rb0["slot"], np.arange(n))
    b.close()
    # same tolerance from here on: rebuild b at tau = 0.05 by forcing the first n queries to miss
    b = oracle.Oracle(None, X.shape[1], 1, cap, 0.05, POL[policy])
    force = np.full(len(Q), -1, np.int32)
    force[:n] = 0
    rb = b.query(Q, force)
    ra = a.query(Q[n:])
    for key in ("hit", "slot", "evicted", "best"):
        assert np.array_equal(ra[key], rb[key][n:]), key
    assert ra["evicted"].max() >= 0 and 0 < ra["hit"].sum() < len(ra["hit"])


def test_fifo_and_lru_traces_differ():
    by = {t["name"]: t for t in all_traces()}
    a, b = by["trace_c2_fifo.txt"], by["trace_c2_lru.txt"]
    assert np.array_equal(a["queries"], b["queries"]) and not np.array_equal(a["hit"], b["hit"])


# ---------------------------------------------------------------- the paper's operation count
def test_flat_probe_operation_count():
    """Section 3.2: with c = 10 000 entries and d = 768 one FLAT lookup performs
    10 000 x 768 = 7.68 million operations."""
    keys = unit_rows(10_000, 768, 11)
    o = oracle.Oracle(None, 768, 1, 10_000, 0.0, oracle.LRU)
    o.cache_load(keys)
    o.query(unit_rows(1, 768, 12))
    assert o.counters()["probe_madds"] == 7_680_000


# ---------------------------------------------------------------- forcing a decision
def test_forced_decisions_follow_the_branch():
    X, Q, _ = small_workload(6, nq=40)
    o = oracle.Oracle(X, X.shape[1], 2, 8, 0.0, oracle.LRU)
    force = np.full(40, -1, np.int32)
    force[5] = 1                                                  # a forced hit returns the nearest key's list
    r = o.query(Q, force)
    assert r["hit"][5] == 1 and np.array_equal(r["ids"][5], r["ids"][r["origin"][5]])
    assert r["hit"].sum() == 1


# ---------------------------------------------------------------- re-ranking factor rho (Section 3.3)
def np_sq(q, rows):
    return ((q.astype(np.float64)[None, :] - rows.astype(np.float64)) ** 2).sum(1)


def test_rho_one_is_the_plain_cache():
    X, Q, _ = small_workload(seed=3)
    a = oracle.Oracle(X, X.shape[1], 5, 10, 0.5, oracle.LRU).query(Q)
    b = oracle.Oracle(X, X.shape[1], 5, 10, 0.5, oracle.LRU, rho=1).query(Q)
    for key in ("ids", "dists", "hit", "slot", "evicted"):
        assert np.array_equal(a[key], b[key])


def test_rho_hand_worked_line():
    """Points on a line, k = 1, rho = 2.  Query 0.0 misses and stores its two nearest points
    (0.1 -> row 0, -0.3 -> row 1) and returns row 0.  Query -0.25 lies within tau of that key:
    among the stored rows the one nearest to -0.25 is row 1 at 0.05^2; without re-ranking the
    stored head, row 0, would come back with the key's own distance 0.1^2."""
    X = np.array([[0.1], [-0.3], [0.9], [-2.0]], np.float32)
    Q = np.array([[0.0], [-0.25]], np.float32)
    r = oracle.Oracle(X, 1, 1, 4, 0.1, oracle.FIFO, rho=2).query(Q)
    assert r["hit"].tolist() == [0, 1]
    assert r["ids"][:, 0].tolist() == [0, 1]
    assert r["dists"][0, 0] == pytest.approx(np.float64(np.float32(0.1)) ** 2, rel=1e-15)
    assert r["dists"][1, 0] == pytest.approx((np.float64(np.float32(-0.25)) - np.float64(np.float32(-0.3))) ** 2, rel=1e-15)
    r1 = oracle.Oracle(X, 1, 1, 4, 0.1, oracle.FIFO, rho=1).query(Q)
    assert r1["ids"][:, 0].tolist() == [0, 0] and r1["dists"][1, 0] == r1["dists"][0, 0]


@pytest.mark.parametrize("rho", [2, 4])
def test_rho_miss_returns_knn_and_hit_reranks_the_stored_rows(rho):
    X, Q, _ = small_workload(seed=5, N=600, nq=200)
    k = 5
    o = oracle.Oracle(X, X.shape[1], k, 4, 0.5, oracle.LRU, rho=rho)      # four entries: topics keep falling out
    r = o.query(Q)
    assert 0.2 < r["hit"].mean() < 0.95
    wide_ids, _ = oracle.exact_topk(X, Q, rho * k)
    for i in range(len(Q)):
        if r["hit"][i] == 0:                                   # the k nearest of the rho k fetched
            full = np_sq(Q[i], X)
            order = np.lexsort((np.arange(len(X)), full))[:k]
            assert np.array_equal(r["ids"][i], order)
            assert np.allclose(r["dists"][i], full[order], rtol=1e-12)
        else:                                                  # the k of the key's rho k rows nearest to THIS query
            stored = wide_ids[r["origin"][i]]
            dd = np_sq(Q[i], X[stored])
            order = np.lexsort((stored, dd))[:k]
            assert np.array_equal(r["ids"][i], stored[order])
            assert np.allclose(r["dists"][i], dd[order], rtol=1e-12)
            # a re-ranked list can never beat the true neighbours of the query
            true = np.sort(np_sq(Q[i], X))[:k]
            assert np.all(r["dists"][i] >= true * (1 - 1e-12))


def test_rho_storing_the_whole_corpus_makes_every_hit_exact():
    """rho * k = N: every key stores all rows, so a re-ranked hit is the exact answer for the
    current query, whatever key matched."""
    X, Q, _ = small_workload(seed=6, N=40, nq=60, topics=5)
    k, rho = 5, 8
    r = oracle.Oracle(X, X.shape[1], k, 6, 1.0, oracle.FIFO, rho=rho).query(Q)
    assert r["hit"].sum() > 10
    ids, dists = oracle.exact_topk(X, Q, k)
    assert np.array_equal(r["ids"], ids) and np.allclose(r["dists"], dists, rtol=1e-12)


def test_rho_duplicate_query_gets_the_head_of_the_stored_list():
    X, Q, _ = small_workload(seed=7)
    Q2 = np.concatenate([Q[:1], Q[:1]])
    r = oracle.Oracle(X, X.shape[1], 4, 5, 0.0, oracle.LRU, rho=3).query(Q2)
    assert r["hit"].tolist() == [0, 1]
    assert np.array_equal(r["ids"][0], r["ids"][1]) and np.array_equal(r["dists"][0], r["dists"][1])


# ---------------------------------------------------------------- PROXIMITY-LSH (Section 3.2)
def planes_for(L, d, seed):
    return np.random.default_rng(seed).standard_normal((L, d)).astype(np.float32)


def test_lsh_hash_is_the_sign_pattern():
    P = planes_for(10, 48, 1)
    for q in unit_rows(50, 48, 2):
        bits = (P.astype(np.float64) @ q.astype(np.float64)) >= 0
        assert oracle.lsh_hash(P, q) == int(sum(1 << l for l in range(10) if bits[l]))
    assert oracle.lsh_hash(P, np.zeros(48, np.float32)) == (1 << 10) - 1          # 0 >= 0 on every plane
    assert oracle.lsh_hash(P[:3], -P[1]) & 2 == 0 and oracle.lsh_hash(P[:3], P[1]) & 2 == 2


@pytest.mark.parametrize("policy", ["lru", "fifo"])
def test_lsh_with_no_hyperplane_is_the_flat_cache(policy):
    X, Q, _ = small_workload(seed=9)
    d = X.shape[1]
    flat = oracle.Oracle(X, d, 5, 12, 0.5, POL[policy]).query(Q)
    lsh = oracle.Oracle(X, d, 5, 12, 0.5, POL[policy], lsh_planes=np.zeros((0, d), np.float32), lsh_bucket=12).query(Q)
    for key in ("ids", "dists", "hit", "slot", "evicted", "best"):
        assert np.array_equal(flat[key], lsh[key])


def test_lsh_buckets_are_independent_flat_caches():
    """Queries are dealt to their buckets; every bucket must behave like a flat cache of b
    entries fed with its own queries alone (own eviction, Section 3.3.2), with slots h*b.."""
    X, Q, _ = small_workload(seed=10, nq=300, topics=40)
    d, L, b = X.shape[1], 3, 2
    P = planes_for(L, d, 4)
    r = oracle.Oracle(X, d, 4, (1 << L) * b, 0.6, oracle.LRU, lsh_planes=P, lsh_bucket=b).query(Q)
    code = np.array([oracle.lsh_hash(P, q) for q in Q])
    assert len(np.unique(code)) >= 4 and r["evicted"].max() >= 0
    for h in np.unique(code):
        sel = np.nonzero(code == h)[0]
        f = oracle.Oracle(X, d, 4, b, 0.6, oracle.LRU).query(Q[sel])
        assert np.array_equal(f["hit"], r["hit"][sel]) and np.array_equal(f["ids"], r["ids"][sel])
        assert np.array_equal(f["slot"] + h * b, r["slot"][sel])
        ev = f["evicted"].copy(); ev[ev >= 0] += h * b
        assert np.array_equal(ev, r["evicted"][sel])


def test_lsh_never_matches_across_buckets_even_with_a_huge_tau():
    X, Q, _ = small_workload(seed=11)
    d = X.shape[1]
    P = planes_for(4, d, 5)
    r = oracle.Oracle(X, d, 3, 16 * 5, 100.0, oracle.FIFO, lsh_planes=P, lsh_bucket=5).query(Q)
    code = np.array([oracle.lsh_hash(P, q) for q in Q])
    first = {}
    for i, h in enumerate(code):
        assert r["hit"][i] == (1 if h in first else 0)                # only the first query of a bucket misses
        first.setdefault(h, i)
        assert r["slot"][i] == h * 5


def test_lsh_operation_count_of_the_papers_example():
    """Section 3.2: c = 10 000, d = 768, b = 20, L = 10: (L + b) d = 23 040 operations per lookup
    once the bucket is full, against 7.68 million for the flat cache."""
    d, L, b = 768, 10, 20
    rng = np.random.default_rng(0)
    base = rng.standard_normal(d).astype(np.float32)
    Q = (base[None, :] + 1e-3 * rng.standard_normal((b + 1, d))).astype(np.float32)   # one bucket, distinct keys
    P = planes_for(L, d, 6)
    assert len({oracle.lsh_hash(P, q) for q in Q}) == 1
    o = oracle.Oracle(None, d, 1, (1 << L) * b, 0.0, oracle.FIFO, lsh_planes=P, lsh_bucket=b)
    o.query(Q[:b])
    before = o.counters()["probe_madds"]
    o.query(Q[b:])
    assert o.counters()["probe_madds"] - before == (L + b) * d == 23040


# ---------------------------------------------------------------- cosine distance (Section 2.2)
def test_cosine_closed_forms():
    e = np.eye(6, dtype=np.float32)
    assert oracle.cosdist(e[0], e[1]) == pytest.approx(1.0, abs=1e-15)           # orthogonal
    assert oracle.cosdist(3 * e[2], 0.25 * e[2]) == 0.0                            # same direction, any length
    assert oracle.cosdist(e[3], -7 * e[3]) == pytest.approx(2.0, abs=1e-15)       # opposite
    a, b = unit_rows(2, 40, 12)
    assert oracle.cosdist(5 * a, 0.1 * b) == pytest.approx(1.0 - float(a.astype(np.float64) @ b.astype(np.float64)), abs=1e-7)
    assert oracle.cosdist(a, a) == 0.0 and oracle.cosdist(a, b) == oracle.cosdist(b, a)


def test_cosine_topk_vs_numpy_and_scale_invariance():
    rng = np.random.default_rng(13)
    X = (rng.standard_normal((500, 24)) * rng.uniform(0.1, 9.0, (500, 1))).astype(np.float32)   # rows of very different length
    Q = rng.standard_normal((7, 24)).astype(np.float32)
    ids, dists = oracle.exact_topk(X, Q, 6, metric=oracle.COSINE)
    Xn = X.astype(np.float64) / np.linalg.norm(X.astype(np.float64), axis=1, keepdims=True)
    for i, q in enumerate(Q):
        qn = q.astype(np.float64) / np.linalg.norm(q.astype(np.float64))
        full = 1.0 - Xn @ qn
        order = np.lexsort((np.arange(len(X)), full))[:6]
        assert np.array_equal(ids[i], order) and np.allclose(dists[i], full[order], atol=1e-12)
    l2_ids, _ = oracle.exact_topk(X, Q, 6)
    assert (l2_ids != ids).any()                                                  # not the Euclidean neighbours here
    ids2, dists2 = oracle.exact_topk(X * np.float32(4.0), Q * np.float32(0.5), 6, metric=oracle.COSINE)
    assert np.array_equal(ids2, ids) and np.allclose(dists2, dists, atol=1e-12)    # powers of two scale exactly


def test_cosine_cache_equals_the_l2_cache_on_unit_vectors():
    """On unit vectors 1 - cos = |a - b|^2 / 2, so the cosine cache at tau must take the decisions
    of the Euclidean cache at 2 tau and return the same lists with half the distances."""
    X, Q, _ = small_workload(seed=14, N=500, nq=150)
    d = X.shape[1]
    c = oracle.Oracle(X, d, 5, 4, 0.25, oracle.LRU, metric=oracle.COSINE).query(Q)
    e = oracle.Oracle(X, d, 5, 4, 0.5, oracle.LRU).query(Q)
    assert 0.2 < c["hit"].mean() < 0.95
    assert np.array_equal(c["hit"], e["hit"]) and np.array_equal(c["ids"], e["ids"]) and np.array_equal(c["slot"], e["slot"])
    assert np.allclose(c["dists"], 0.5 * e["dists"], rtol=1e-5)


def test_cosine_duplicate_hits_at_tau_zero_whatever_its_length():
    X, Q, _ = small_workload(seed=15)
    Q2 = np.concatenate([Q[:1], 2 * Q[:1], Q[1:2]])
    r = oracle.Oracle(X, X.shape[1], 3, 4, 0.0, oracle.FIFO, metric=oracle.COSINE).query(Q2)
    assert r["hit"].tolist() == [0, 1, 0]


# ---------------------------------------------------------------- inner product (Section 2.2)
def test_inner_product_closed_forms():
    assert oracle.ipdist([1, 2, 3], [4, 5, 6]) == -32.0
    e = np.eye(5, dtype=np.float32)
    for i in range(5):
        for j in range(5):
            assert oracle.ipdist(e[i], e[j]) == (-1.0 if i == j else 0.0)
    a, b = unit_rows(2, 64, 21)
    assert oracle.ipdist(a, b) == oracle.ipdist(b, a)
    assert oracle.ipdist(a, -a) == pytest.approx(1.0, abs=1e-6) and oracle.ipdist(a, -a) > 0      # opposite: the farthest
    assert oracle.ipdist(2 * a, b) == pytest.approx(2 * oracle.ipdist(a, b), rel=1e-15)           # linear, unlike a true distance
    assert oracle.ipdist([3, 0], [0, 4]) == 0.0 and oracle.sqdist([3, 0], [0, 4]) == 25.0          # not the Euclidean value


def test_inner_product_topk_vs_numpy():
    rng = np.random.default_rng(22)
    X = (rng.standard_normal((600, 40)) * rng.uniform(0.2, 3.0, (600, 1))).astype(np.float32)
    Q = rng.standard_normal((6, 40)).astype(np.float32)
    X[77] = X[12]                                                     # equal inner products: the lower id first
    ids, dists = oracle.exact_topk(X, Q, 600, metric=oracle.IP)
    for i, q in enumerate(Q):
        full = -(X.astype(np.float64) @ q.astype(np.float64))
        order = np.lexsort((np.arange(len(X)), full))
        p12, p77 = np.where(ids[i] == 12)[0][0], np.where(ids[i] == 77)[0][0]
        assert p77 == p12 + 1
        assert np.array_equal(ids[i][:10], order[:10]) and np.allclose(dists[i], np.sort(full), rtol=0, atol=1e-12)
        assert np.all(np.diff(dists[i]) >= 0) and dists[i][0] < 0    # most similar first
    l2_ids, _ = oracle.exact_topk(X, Q, 10)
    assert (l2_ids != ids[:, :10]).any()                              # rows of unequal length: not the Euclidean neighbours


def test_inner_product_equals_euclidean_neighbours_on_unit_vectors():
    """|q - x|^2 = |q|^2 + |x|^2 - 2 q.x: with all lengths equal the two rankings agree."""
    X, Q = unit_rows(800, 48, 23), unit_rows(9, 48, 24)
    ip_ids, ip_d = oracle.exact_topk(X, Q, 12, metric=oracle.IP)
    l2_ids, l2_d = oracle.exact_topk(X, Q, 12)
    assert np.array_equal(ip_ids, l2_ids)
    assert np.allclose(ip_d, (l2_d - 2.0) / 2.0, atol=2e-7)


def test_inner_product_cache_follows_algorithm_1():
    """Independent replay with -q.k as the distance; the tolerance is negative here (a key matches
    when q.k >= 0.9), which only this metric allows."""
    X, Q, _ = small_workload(16, nq=200)
    cap, tau = 6, -0.9
    r = oracle.Oracle(X, X.shape[1], 3, cap, tau, oracle.LRU, metric=oracle.IP).query(Q)
    keys, stamp = {}, {}
    Q64 = Q.astype(np.float64)
    for i in range(len(Q)):
        dist = {s: -float(Q64[i] @ Q64[j]) for s, j in keys.items()}
        best = min(dist, key=lambda s: (dist[s], s)) if dist else None
        if best is not None and dist[best] <= tau:
            assert r["hit"][i] == 1 and r["slot"][i] == best and r["origin"][i] == keys[best]
            assert r["best"][i] == pytest.approx(dist[best], abs=1e-12)
            stamp[best] = i
        else:
            assert r["hit"][i] == 0
            if len(keys) >= cap:
                victim = min(stamp, key=stamp.get)
                assert r["evicted"][i] == victim
                del keys[victim], stamp[victim]
                slot = victim
            else:
                slot = len(keys)
            assert r["slot"][i] == slot
            keys[slot], stamp[slot] = i, i
    assert 0.1 < r["hit"].mean() < 0.95 and (r["evicted"] >= 0).any()
    ids, dists = oracle.exact_topk(X, Q, 3, metric=oracle.IP)
    miss = r["hit"] == 0
    assert np.array_equal(r["ids"][miss], ids[miss]) and np.array_equal(r["dists"][miss], dists[miss])


def test_inner_product_prefers_the_longer_key_and_tau_zero_is_a_half_space():
    e = np.eye(4, dtype=np.float32)
    keys = np.stack([e[0], 3 * e[0], -e[0]])
    o = oracle.Oracle(None, 4, 1, 3, 0.0, oracle.FIFO, metric=oracle.IP)
    o.cache_load(keys)
    r = o.query(np.stack([e[0], e[1], -e[0] + e[1]]))
    assert r["slot"].tolist()[0] == 1 and r["best"][0] == -3.0      # not its own duplicate in slot 0
    assert r["hit"].tolist() == [1, 1, 1]                           # e1 is orthogonal to every key: -0 <= 0 matches (slot 0)
    assert r["slot"].tolist()[1] == 0 and r["slot"].tolist()[2] == 2
    o2 = oracle.Oracle(None, 4, 1, 3, -0.5, oracle.FIFO, metric=oracle.IP)
    o2.cache_load(keys)
    assert o2.query(np.stack([e[1]]))["hit"].tolist() == [0]        # inner product 0 < 0.5


def test_negative_tolerance_goes_with_the_inner_product_only():
    with pytest.raises(ValueError):
        oracle.Oracle(None, 8, 1, 4, -0.1, oracle.LRU)
    with pytest.raises(ValueError):
        oracle.Oracle(None, 8, 1, 4, -0.1, oracle.LRU, metric=oracle.COSINE)
    with pytest.raises(ValueError):
        oracle.Oracle(None, 8, 1, 4, float("nan"), oracle.LRU, metric=oracle.IP)
    with pytest.raises(ValueError):                                   # hyperplane buckets are for angles
        oracle.Oracle(None, 8, 1, 8, 0.5, oracle.LRU, lsh_planes=np.zeros((1, 8), np.float32), lsh_bucket=4, metric=oracle.IP)
    oracle.Oracle(None, 8, 1, 4, -0.1, oracle.LRU, metric=oracle.IP).close()
