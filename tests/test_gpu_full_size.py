"""Parity at the full sizes of the benchmark workloads, in the launch configuration bench.py times.

The oracle cannot answer every miss at 24 million or 100 million rows, so the check is split the
way the method allows: hit / miss decisions, matched keys and evictions depend on the query stream
alone, so the oracle replays the whole prefix of the stream without a corpus and every flag is
compared; a hit must return exactly the list of the miss that created its key (checked on the GPU
output itself); and for a seeded sample of misses the oracle computes the exact k nearest rows from
the corpus bytes copied off the device in chunks."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05530_b200 import prox, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
POL = {"lru": oracle.LRU, "fifo": oracle.FIFO}


def run_full_size(cfg, runs, seed=0, chunk_rows=1 << 20, lsh=None):
    """runs: (tau, batches, sampled misses) per tolerance, all on one copy of the corpus; the sampled
    misses of all runs share one pass of the oracle over the corpus bytes.
    lsh = (L, b): PROXIMITY-LSH with 2^L buckets of b entries instead of the flat cache of cfg.capacity."""
    need = cfg.N * cfg.d * 6 + (8 << 30)
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip(f"needs {need >> 30} GB of device memory")
    corpus = W.make_corpus(cfg.N, cfg.d, cfg.n_components, seed, DEV)
    n_max = max(nb for _, nb, _ in runs) * cfg.batch
    queries, _, _ = W.make_query_stream(corpus, n_max, cfg.n_topics, cfg.zipf_s, cfg.sigma, seed)
    Q = queries.cpu().numpy()
    capacity, planes, bucket = cfg.capacity, None, 0
    if lsh is not None:
        planes = torch.randn(lsh[0], cfg.d, generator=torch.Generator().manual_seed(seed + 3))
        bucket, capacity = lsh[1], (1 << lsh[0]) * lsh[1]
    results, checks = [], []
    for tau, n_batches, n_samples in runs:
        n = n_batches * cfg.batch
        p = prox.Prox(corpus, cfg.k, capacity, tau, cfg.policy, lsh_planes=None if planes is None else planes.to(DEV),
                      lsh_bucket=bucket)
        ids = torch.empty(n, cfg.k, dtype=torch.int64, device=DEV)
        dists = torch.empty(n, cfg.k, dtype=torch.float32, device=DEV)
        hit = torch.empty(n, dtype=torch.uint8, device=DEV)
        for a in range(0, n, cfg.batch):
            p.query_batch(queries[a:a + cfg.batch], ids[a:a + cfg.batch], dists[a:a + cfg.batch], hit[a:a + cfg.batch])
        torch.cuda.synchronize()
        assert p.status() == prox.OK, prox.last_error()
        stats = p.stats()
        p.close()
        ids, dists, hit = ids.cpu().numpy(), dists.cpu().numpy(), hit.cpu().numpy()

        # 1. the cache trace of the whole prefix (needs no corpus)
        o = oracle.Oracle(None, cfg.d, cfg.k, capacity, float(np.float32(tau)), POL[cfg.policy],
                          lsh_planes=None if planes is None else planes.numpy(), lsh_bucket=bucket)
        r = o.query(Q[:n])
        o.close()
        assert np.array_equal(hit, r["hit"]), f"tau {tau}: first differing flag at query {np.nonzero(hit != r['hit'])[0][0]}"
        assert stats["hits"] == int(r["hit"].sum()) and stats["evictions"] == int((r["evicted"] >= 0).sum())
        assert stats["unresolved"] == 0

        # 2. a hit returns the list of the miss that made its key
        for i in np.nonzero(r["hit"] == 1)[0]:
            src = int(r["origin"][i])
            assert np.array_equal(ids[i], ids[src]) and np.array_equal(dists[i], dists[src])

        # every miss list is sorted and made of valid, distinct rows
        misses = np.nonzero(r["hit"] == 0)[0]
        m_ids = ids[misses]
        assert m_ids.min() >= 0 and m_ids.max() < cfg.N
        assert all(len(set(row)) == cfg.k for row in m_ids[:: max(1, len(m_ids) // 500)])
        assert np.all(np.diff(dists[misses], axis=1) >= 0)

        # 3. a seeded sample of the misses for the oracle's exact top-k (computed below)
        rng = np.random.default_rng(seed + int(round(tau * 1000)))
        sample = np.sort(rng.choice(misses, size=min(n_samples, len(misses)), replace=False))
        checks.append((tau, sample, [oracle.ChunkedTopK(Q[i], cfg.k) for i in sample], ids, dists))
        results.append(dict(tau=tau, hit_rate=float(r["hit"].mean()), stats=stats, misses_per_batch=len(misses) / n_batches))

    stage = torch.empty(chunk_rows, cfg.d, dtype=torch.float32).pin_memory()
    for r0 in range(0, cfg.N, chunk_rows):
        rows = min(chunk_rows, cfg.N - r0)
        stage[:rows].copy_(corpus[r0:r0 + rows])
        chunk = stage[:rows].numpy()
        for _, _, tops, _, _ in checks:
            for t in tops:
                t.feed(chunk)
    for tau, sample, tops, ids, dists in checks:
        for i, t in zip(sample, tops):
            assert np.array_equal(ids[i], t.ids), f"tau {tau}: ids differ at sampled miss {i}"
            assert np.allclose(dists[i], t.dists, rtol=1e-4, atol=1e-12)
    return results


def test_one_million_rows_batch64_lru_full_size():
    cfg = W.CONFIGS["1m"]
    res = run_full_size(cfg, [(0.5, 100, 24), (0.0, 20, 16), (1.0, 40, 8)])
    assert 0.3 < res[0]["hit_rate"] < 0.95 and res[0]["stats"]["evictions"] > 0
    assert res[1]["hit_rate"] == 0.0


def test_one_million_rows_lsh_full_size():
    cfg = W.CONFIGS["1m"]
    res = run_full_size(cfg, [(0.5, 60, 12)], lsh=(8, 4))
    assert 0.2 < res[0]["hit_rate"] < 0.95 and res[0]["stats"]["evictions"] > 0


def test_24m_rows_batch256_lru_full_size():
    """tau = 0 and 0.5: every launch of the scan carries 256 misses, the shape the benchmark's headline
    times; tau = 1.0: launches of 50 to 100 misses once the cache has warmed up."""
    cfg = W.CONFIGS["large"]
    res = run_full_size(cfg, [(0.0, 6, 32), (0.5, 6, 32), (1.0, 24, 16)])
    assert res[0]["hit_rate"] == 0.0 and res[0]["misses_per_batch"] == 256
    assert res[1]["misses_per_batch"] > 250
    assert 0.2 < res[2]["hit_rate"] < 0.95


def test_100m_rows_d128_batch1024_fifo_full_size():
    cfg = W.CONFIGS["lowhit"]
    res = run_full_size(cfg, [(0.3, 4, 32)])
    assert res[0]["hit_rate"] < 0.5
