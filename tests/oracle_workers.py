"""Oracle runs that take minutes, moved to worker processes so that they overlap one another and the
GPU side of a test.  The workers are started with the `spawn` method (a process forked after the
first CUDA call is not safe) and import nothing but numpy and the oracle; inputs travel through
shared memory by name, results come back as small arrays."""
from __future__ import annotations

import multiprocessing as mp
from multiprocessing import shared_memory

import numpy as np


def share(a: np.ndarray):
    """Copy an array into a new shared-memory block; returns (block, descriptor for the worker)."""
    a = np.ascontiguousarray(a)
    blk = shared_memory.SharedMemory(create=True, size=max(1, a.nbytes))
    np.ndarray(a.shape, a.dtype, buffer=blk.buf)[...] = a
    return blk, (blk.name, a.shape, a.dtype.str)


def _attach(desc):
    name, shape, dtype = desc
    blk = shared_memory.SharedMemory(name=name)
    return blk, np.ndarray(shape, np.dtype(dtype), buffer=blk.buf)


def probe_trace_worker(keys_desc, batches_desc, tau, policy):
    """Cache loaded with the keys, then the batches one query after the other (no corpus: the cache
    trace depends on the query stream alone).  Returns hit, slot, best and evicted per batch."""
    import oracle
    kb, keys = _attach(keys_desc)
    qb, batches = _attach(batches_desc)
    try:
        o = oracle.Oracle(None, keys.shape[1], 1, keys.shape[0], float(np.float32(tau)),
                          oracle.LRU if policy == "lru" else oracle.FIFO)
        o.cache_load(keys)
        out = []
        for Q in batches:
            r = o.query(Q)
            out.append(dict(hit=r["hit"], slot=r["slot"], best=r["best"], evicted=r["evicted"]))
        o.close()
        return out
    finally:
        del keys, batches
        kb.close()
        qb.close()


def pool(n: int):
    return mp.get_context("spawn").Pool(n)
