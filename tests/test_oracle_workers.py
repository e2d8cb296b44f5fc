"""The worker-process harness of the long oracle runs returns what a direct call returns."""
import numpy as np

import oracle
import oracle_workers
from paper_2503_05530_b200 import workloads as W


def test_probe_trace_worker_equals_a_direct_run():
    keys, centres = W.make_probe_keys(300, 32, 16, seed=3)
    Qs = np.stack([W.make_probe_batch(keys, centres, 40, 0.02, 3, b).numpy() for b in range(2)])
    kb, kdesc = oracle_workers.share(keys.numpy())
    qb, qdesc = oracle_workers.share(Qs)
    try:
        with oracle_workers.pool(2) as pool:
            jobs = {pol: pool.apply_async(oracle_workers.probe_trace_worker, (kdesc, qdesc, 0.5, pol)) for pol in ("lru", "fifo")}
            got = {pol: j.get(timeout=120) for pol, j in jobs.items()}
    finally:
        for blk in (kb, qb):
            blk.close()
            blk.unlink()
    for pol in ("lru", "fifo"):
        o = oracle.Oracle(None, 32, 1, 300, float(np.float32(0.5)), oracle.LRU if pol == "lru" else oracle.FIFO)
        o.cache_load(keys.numpy())
        for b in range(2):
            r = o.query(Qs[b])
            for key in ("hit", "slot", "best", "evicted"):
                assert np.array_equal(got[pol][b][key], r[key])
