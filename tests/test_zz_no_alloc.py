"""The allocation-free lookup (prox_nearest_key_static) against the regular probe.

Some users of this library run where device memory cannot be allocated at call time (inside an
application that owns the whole memory pool, or under a fixed memory budget).  For them the library
has one entry point whose only scratch is an array built into the library image.  This test calls
it through the C ABI twice in a row, on different queries, and checks both answers against
prox_probe_batch on a cache that holds the same keys, and against the CPU oracle (a cache loaded
with the keys and a tolerance so large that every query hits: the matched slot and the distance to
it are the nearest key and its distance): the second call sees the scratch as the first one left
it, so a stale counter or partial result would show up there.  The file sorts last on
purpose: a run that stops at the first failure has then already run every other test."""
import numpy as np
import pytest
import torch

import oracle
from paper_2503_05530_b200 import prox, workloads as W

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def reference_nearest(keys_d, queries_d, policy="fifo"):
    """Nearest slot and distance from the existing entry point: a cache pre-filled with the keys and a
    tolerance so large that every query hits its nearest key (FIFO: hits change nothing)."""
    p = prox.Prox(keys_d[:64].contiguous(), 1, keys_d.shape[0], 1.0e9, policy)
    p.cache_load(keys_d)
    hit, slot, dist = p.probe_batch(queries_d)
    torch.cuda.synchronize()
    assert p.status() == prox.OK and bool(hit.all())
    p.close()
    return slot.cpu().numpy(), dist.cpu().numpy()


def oracle_nearest(keys, queries):
    """The same two numbers from the oracle: FIFO, so the hits leave the cache as it was loaded."""
    o = oracle.Oracle(None, keys.shape[1], 1, keys.shape[0], 1.0e9, oracle.FIFO)
    o.cache_load(keys.numpy())
    r = o.query(queries.numpy())
    o.close()
    assert r["hit"].all()
    return r["slot"], r["best"]


def test_static_scratch_lookup_matches_probe_on_two_calls_in_a_row():
    keys, centres = W.make_probe_keys(5003, 256, 64, seed=21)
    keys_d = keys.to(DEV)
    out_slot = torch.empty(256, dtype=torch.int32, device=DEV)
    out_dist = torch.empty(256, dtype=torch.float32, device=DEV)
    for call, B in enumerate([256, 77]):                       # full and ragged batch, back to back
        Qc = W.make_probe_batch(keys, centres, 256, 0.02, 21, call)[:B].contiguous()
        Q = Qc.to(DEV)
        out_slot.fill_(-7)
        out_dist.fill_(-1.0)
        prox.nearest_key_static(keys_d, Q, out_slot, out_dist)
        torch.cuda.synchronize()
        ref_slot, ref_dist = reference_nearest(keys_d, Q)
        assert np.array_equal(out_slot[:B].cpu().numpy(), ref_slot)
        assert np.allclose(out_dist[:B].cpu().numpy(), ref_dist, rtol=1e-6, atol=0)
        o_slot, o_dist = oracle_nearest(keys, Qc)
        assert np.array_equal(out_slot[:B].cpu().numpy(), o_slot)
        assert np.allclose(out_dist[:B].cpu().numpy(), o_dist, rtol=1e-6, atol=0)
        assert (out_slot[B:] == -7).all()                       # nothing written past the batch


def test_static_scratch_lookup_rejects_sizes_beyond_its_scratch():
    lib = prox.load_library()
    k = torch.zeros(8, 16, device=DEV)
    q = torch.zeros(300, 16, device=DEV)
    s = torch.empty(300, dtype=torch.int32, device=DEV)
    dd = torch.empty(300, dtype=torch.float32, device=DEV)
    assert lib.prox_nearest_key_static(k.data_ptr(), 8, 16, q.data_ptr(), 257, s.data_ptr(), dd.data_ptr(), None) == prox.ERR_INVALID_ARG
    assert "256" in prox.last_error()
    assert lib.prox_nearest_key_static(k.data_ptr(), (1 << 22) + 1, 16, q.data_ptr(), 4, s.data_ptr(), dd.data_ptr(), None) == prox.ERR_INVALID_ARG
    assert lib.prox_nearest_key_static(None, 8, 16, q.data_ptr(), 4, s.data_ptr(), dd.data_ptr(), None) == prox.ERR_INVALID_ARG
