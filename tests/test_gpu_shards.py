"""A corpus split by rows: G shard handles (here all on one GPU, their kernels simply run one after
the other: none waits for another) must give, after the exchange and the merge, exactly what the
oracle gives on the whole corpus, and every replica the same bytes."""
import numpy as np
import pytest
import torch

from paper_2503_05530_b200 import prox, workloads as W
from parity import compare

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_shards(X, Q, k, cap, tau, policy, batch, n_shards, metric="l2", order=None):
    """Returns (ids, dists, hit, stats) of replica 0 after checking that all replicas agree."""
    Xd, Qd = X.to(DEV), Q.to(DEV)
    N = X.shape[0]
    shards = []
    for g in range(n_shards):
        first, cnt = prox.shard_rows(N, n_shards, g)
        shards.append(prox.ProxShard(Xd[first:first + cnt].contiguous(), first, N, k, cap, tau, policy, metric=metric))
    try:
        n = Q.shape[0]
        outs = [(torch.empty(n, k, dtype=torch.int64, device=DEV), torch.empty(n, k, dtype=torch.float32, device=DEV),
                 torch.empty(n, dtype=torch.uint8, device=DEV)) for _ in shards]
        for a in range(0, n, batch):
            b = min(n, a + batch)
            recs = []
            for sh, (ids, dists, hit) in zip(shards, outs):
                rec = torch.empty(sh.exchange_bytes(b - a), dtype=torch.uint8, device=DEV)
                sh.shard_scan(Qd[a:b], ids[a:b], dists[a:b], hit[a:b], rec)
                recs.append(rec)
            for r, (sh, (ids, dists, hit)) in enumerate(zip(shards, outs)):
                # every replica may receive the records in another order
                perm = list(range(n_shards)) if order is None else list(np.roll(order, r))
                gathered = torch.cat([recs[g] for g in perm])
                sh.shard_merge(Qd[a:b], gathered, n_shards, ids[a:b], dists[a:b])
        torch.cuda.synchronize()
        stats = []
        for sh in shards:
            assert sh.status() == prox.OK, prox.last_error()
            stats.append(sh.stats())
    finally:
        for sh in shards:
            sh.close()
    res = [tuple(t.cpu().numpy() for t in o) for o in outs]
    for r in range(1, n_shards):
        for x, y in zip(res[0], res[r]):
            assert x.tobytes() == y.tobytes(), f"replica {r} differs from replica 0"
        for key in ("queries", "hits", "misses", "intra_batch_hits", "evictions", "count"):
            assert stats[r][key] == stats[0][key]
    return res[0] + (stats[0],)


@pytest.mark.parametrize("policy,batch,n_shards,k", [("lru", 64, 3, 10), ("fifo", 1, 2, 5), ("lru", 300, 5, 32),
                                                     ("lru", 1000, 8, 64)])
def test_row_shards_match_the_oracle_on_the_whole_corpus(policy, batch, n_shards, k):
    X = W.make_corpus(30011, 128, 64, 5)                      # a row count no shard count divides
    Q, _, _ = W.make_query_stream(X, 1500, 300, 1.0, 0.05, 5)
    gpu = run_shards(X, Q, k, 200, 0.55, policy, batch, n_shards, order=list(range(n_shards))[::-1])
    r = compare(X.numpy(), Q.numpy(), k, 200, 0.55, policy, gpu)
    assert 0.1 < r["hit_rate"] < 0.95
    assert gpu[3]["intra_batch_hits"] > 0 or batch == 1


def test_one_shard_equals_the_unsharded_handle():
    X = W.make_corpus(20000, 256, 64, 6)
    Q, _, _ = W.make_query_stream(X, 600, 150, 1.0, 0.05, 6)
    ids, dists, hit, stats = run_shards(X, Q, 16, 100, 1.2, "lru", 128, 1)
    with prox.Prox(X.to(DEV), 16, 100, 1.2, "lru") as p:
        ids1 = torch.empty(600, 16, dtype=torch.int64, device=DEV)
        d1 = torch.empty(600, 16, dtype=torch.float32, device=DEV)
        h1 = torch.empty(600, dtype=torch.uint8, device=DEV)
        for a in range(0, 600, 128):
            p.query_batch(Q[a:a + 128].to(DEV), ids1[a:a + 128], d1[a:a + 128], h1[a:a + 128])
        torch.cuda.synchronize()
    assert np.array_equal(ids, ids1.cpu().numpy()) and np.array_equal(hit, h1.cpu().numpy())
    assert dists.tobytes() == d1.cpu().numpy().tobytes()


def test_row_shards_cosine_distance():
    X = W.make_corpus(12007, 64, 32, 7) * 3.0
    Q, _, _ = W.make_query_stream(X, 800, 200, 1.0, 0.05, 7)
    Q = Q * torch.linspace(0.5, 2.0, Q.shape[0])[:, None]     # lengths must not matter
    gpu = run_shards(X, Q, 8, 64, 0.05, "lru", 100, 4, metric="cosine")
    r = compare(X.numpy(), Q.numpy(), 8, 64, 0.05, "lru", gpu, metric="cosine")
    assert 0.05 < r["hit_rate"] < 0.98


def test_row_shards_inner_product():
    X = W.make_corpus(24001, 64, 32, 12)
    Q, _, _ = W.make_query_stream(X, 900, 120, 1.0, 0.04, 12)
    X = (X * (0.5 + 1.5 * torch.rand(X.shape[0], 1, generator=torch.Generator().manual_seed(13)))).contiguous()
    gpu = run_shards(X, Q, 8, 64, -0.9, "lru", 100, 4, metric="ip")
    r = compare(X.numpy(), Q.numpy(), 8, 64, -0.9, "lru", gpu, metric="ip")
    assert 0.05 < r["hit_rate"] < 0.98


def test_duplicate_rows_across_shards_keep_the_lower_id():
    base = W.make_corpus(4000, 64, 16, 8)
    X = torch.cat([base, base, base])                          # every row three times, one copy per shard
    Q, _, _ = W.make_query_stream(base, 200, 50, 1.0, 0.05, 8)
    ids, dists, hit, _ = run_shards(X, Q, 6, 32, 0.0, "lru", 50, 3)
    miss = hit == 0
    # the three copies of a row are at the same distance: they come out in order of their ids
    assert miss.any()
    got = ids[miss]
    assert np.array_equal(got[:, 1] - got[:, 0], np.full(miss.sum(), 4000))
    assert np.array_equal(got[:, 2] - got[:, 1], np.full(miss.sum(), 4000))
    compare(X.numpy(), Q.numpy(), 6, 32, 0.0, "lru", (ids, dists, hit, _))


def test_shard_argument_checks():
    X = W.make_corpus(1000, 32, 8, 9).to(DEV)
    lib = prox.load_library()
    assert not lib.prox_create_shard(X.data_ptr(), 1000, 32, 4, 10, 0.5, 0, 0, 5, 1004)
    assert "row_offset" in prox.last_error()
    with prox.ProxShard(X, 0, 1000, 4, 10, 0.5) as sh:
        q = X[:8].contiguous()
        ids = torch.empty(8, 4, dtype=torch.int64, device=DEV)
        dists = torch.empty(8, 4, dtype=torch.float32, device=DEV)
        hit = torch.empty(8, dtype=torch.uint8, device=DEV)
        assert sh.exchange_bytes(8) == 16 * 8 * 4 and sh.exchange_bytes(0) == 0
        with pytest.raises(prox.ProxError, match="prox_shard_scan"):
            prox.Prox.query_batch(sh, q, ids, dists, hit)
        rec = torch.empty(sh.exchange_bytes(8), dtype=torch.uint8, device=DEV)
        with pytest.raises(prox.ProxError, match="waiting"):
            sh.shard_merge(q, rec, 1, ids, dists)
        sh.shard_scan(q, ids, dists, hit, rec)
        with pytest.raises(prox.ProxError, match="not completed"):
            sh.shard_scan(q, ids, dists, hit, rec)
        rc = lib.prox_shard_merge(sh._h, q.data_ptr(), 8, rec.data_ptr(), 33, ids.data_ptr(), dists.data_ptr(), None)
        assert rc == prox.ERR_INVALID_ARG and "G must" in prox.last_error()
        sh.shard_merge(q, rec, 1, ids, dists)
        torch.cuda.synchronize()
        assert sh.status() == prox.OK
    with prox.Prox(X, 4, 10, 0.5) as p:
        rc = lib.prox_shard_scan(p._h, X.data_ptr(), 8, ids.data_ptr(), dists.data_ptr(), hit.data_ptr(),
                                 rec.data_ptr(), None)
        assert rc == prox.ERR_INVALID_ARG and "not a shard handle" in prox.last_error()
