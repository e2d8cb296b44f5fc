"""Shared helpers of the GPU parity tests: run a stream through the CUDA library and through the
oracle on the same bytes, and compare under the stated rule.

Rule: hit flags and returned ids equal; distances within 1e-4 relative.  A query may differ only
if (i) its nearest-key distance ties with tau to 1e-5 relative (never when that distance is 0),
or (ii) its k-th and (k+1)-th neighbour distances, or two neighbours inside the list, tie to 1e-5
relative, and the ids that differ are exactly the tied ones.  Such queries are counted and must
stay below 0.1 % of the stream; unless a test says otherwise none is accepted at all."""
import numpy as np
import torch

import oracle
from paper_2503_05530_b200 import prox

POL = {"lru": oracle.LRU, "fifo": oracle.FIFO}
ORACLE_METRIC = {"l2": oracle.L2SQ, "cosine": oracle.COSINE, "ip": oracle.IP}
REL_TIE = 1e-5
REL_DIST = 1e-4


def run_gpu(corpus_t, queries_t, k, capacity, tau, policy, batch, scan_mode=None, host_api=False, rho=1,
            lsh_planes=None, lsh_bucket=0, metric="l2", recorded=False):
    """corpus_t, queries_t: CUDA float32 tensors.  Returns numpy (ids, dists, hit) and the stats."""
    planes_t = None if lsh_planes is None else torch.as_tensor(lsh_planes).to(corpus_t.device)
    p = prox.Prox(corpus_t, k, capacity, tau, policy, rho=rho, lsh_planes=planes_t, lsh_bucket=lsh_bucket, metric=metric)
    try:
        if scan_mode is not None:
            p.set_scan_mode(scan_mode)
        n = queries_t.shape[0]
        ids = torch.empty(n, k, dtype=torch.int64, device=corpus_t.device)
        dists = torch.empty(n, k, dtype=torch.float32, device=corpus_t.device)
        hit = torch.empty(n, dtype=torch.uint8, device=corpus_t.device)
        if host_api:
            qh = queries_t.cpu().pin_memory()
            ih, dh, hh = ids.cpu().pin_memory(), dists.cpu().pin_memory(), hit.cpu().pin_memory()
            for a in range(0, n, batch):
                b = min(n, a + batch)
                p.query_batch_host(qh[a:b], ih[a:b], dh[a:b], hh[a:b])
            ids, dists, hit = ih, dh, hh
        elif recorded:
            # the batch call recorded once on fixed buffers and replayed for every full batch; a ragged
            # last batch takes the plain call on the same stream
            dev = corpus_t.device
            qb = torch.empty(batch, queries_t.shape[1], dtype=torch.float32, device=dev)
            ib = torch.empty(batch, k, dtype=torch.int64, device=dev)
            db = torch.empty(batch, k, dtype=torch.float32, device=dev)
            hb = torch.empty(batch, dtype=torch.uint8, device=dev)
            side = torch.cuda.Stream(device=dev)
            side.wait_stream(torch.cuda.current_stream(dev))
            with torch.cuda.stream(side):
                rec = p.record_batch(qb, ib, db, hb, stream=side)
                for a in range(0, n, batch):
                    b = min(n, a + batch)
                    if b - a == batch:
                        qb.copy_(queries_t[a:b])
                        rec.replay(stream=side)
                        ids[a:b].copy_(ib); dists[a:b].copy_(db); hit[a:b].copy_(hb)
                    else:
                        p.query_batch(queries_t[a:b], ids[a:b], dists[a:b], hit[a:b], stream=side)
                side.synchronize()
                rec.close()
        else:
            for a in range(0, n, batch):
                b = min(n, a + batch)
                p.query_batch(queries_t[a:b], ids[a:b], dists[a:b], hit[a:b])
        torch.cuda.synchronize()
        assert p.status() == prox.OK, prox.last_error()
        stats = p.stats()
    finally:
        p.close()
    return ids.cpu().numpy(), dists.cpu().numpy(), hit.cpu().numpy(), stats


def run_oracle(corpus, queries, k, capacity, tau, policy, gpu_hit=None, max_forced=16, rho=1, lsh_planes=None,
               lsh_bucket=0, metric="l2"):
    """Oracle on the same bytes.  tau is rounded to float32 first, as the C ABI takes a float.
    If gpu_hit is given, queries whose decision ties with tau (rule (i)) adopt the GPU's
    decision so that both state machines stay in step; returns the list of such queries."""
    tau32 = float(np.float32(tau))
    d = queries.shape[1]
    force = np.full(len(queries), -1, np.int32)
    forced = []
    while True:
        o = oracle.Oracle(corpus, d, k, capacity, tau32, POL[policy], rho=rho, lsh_planes=lsh_planes, lsh_bucket=lsh_bucket,
                          metric=ORACLE_METRIC[metric])
        r = o.query(queries, force)
        o.close()
        if gpu_hit is None:
            return r, forced
        diff = np.nonzero(r["hit"] != gpu_hit)[0]
        if len(diff) == 0 or len(forced) >= max_forced:
            return r, forced
        i = int(diff[0])
        best = r["best"][i]
        tie = best != 0.0 and np.isfinite(best) and abs(best - tau32) < REL_TIE * max(abs(tau32), abs(best))
        if not tie:
            return r, forced
        force[i] = int(gpu_hit[i])
        forced.append(i)


def ids_differ_only_within_ties(corpus, q, gpu_ids, ref_ids, ref_dists, metric="l2"):
    """Rule (ii), applied to the positions that differ and to nothing else: wherever the library's
    list names another row than the oracle's, that row's exact distance to the query must tie with
    the oracle's distance at the same position to 1e-5 relative (two rows swapped inside the
    list, or another row of a tie group at the k / k+1 boundary), and the library's list must not
    name a row twice.  A tie somewhere else in the list excuses nothing."""
    if len(set(int(x) for x in gpu_ids)) != len(gpu_ids):
        return False
    dist = {"cosine": oracle.cosdist, "ip": oracle.ipdist}.get(metric, oracle.sqdist)
    for p in np.nonzero(np.asarray(gpu_ids) != np.asarray(ref_ids))[0]:
        g = int(gpu_ids[p])
        if g < 0 or g >= corpus.shape[0]:
            return False
        dg, dr = dist(q, corpus[g]), float(ref_dists[p])
        if not abs(dg - dr) < REL_TIE * max(abs(dr), abs(dg), 1e-300):
            return False
    return True


def compare(corpus, queries, k, capacity, tau, policy, gpu, max_excused_frac=1e-3, rho=1, lsh_planes=None, lsh_bucket=0,
            metric="l2", allow_excused=False):
    """allow_excused=False (the default): the exemptions exist but no query may need one -- probe,
    threshold test and rerank run in fp64 like the oracle, so none has ever been needed; a test
    whose inputs are built to tie passes allow_excused=True and stays under max_excused_frac."""
    ids, dists, hit, stats = gpu
    ref, forced = run_oracle(corpus, queries, k, capacity, tau, policy, gpu_hit=hit, rho=rho, lsh_planes=lsh_planes,
                             lsh_bucket=lsh_bucket, metric=metric)
    n = len(queries)
    bad_hit = np.nonzero(ref["hit"] != hit)[0]
    assert len(bad_hit) == 0, f"hit/miss differs first at query {bad_hit[0]} (best={ref['best'][bad_hit[0]]}, tau={tau})"
    excused = set(forced)
    rows_bad = np.nonzero((ref["ids"] != ids).any(axis=1))[0]
    for i in rows_bad:
        origin = int(ref["origin"][i])                       # the miss whose list is returned
        src = origin if origin >= 0 else i
        # a re-ranked hit is measured against the current query, everything else against the query of the list
        q_eval = queries[i] if (rho > 1 and src != i) else queries[src]
        tie = ids_differ_only_within_ties(corpus, q_eval, ids[i], ref["ids"][i], ref["dists"][i], metric)
        assert tie, f"ids differ at query {i} (list of query {src}): oracle {ref['ids'][i]} gpu {ids[i]}"
        excused.add(int(i))
    ok_rows = np.setdiff1d(np.arange(n), rows_bad)
    rd, gd = ref["dists"][ok_rows], dists[ok_rows].astype(np.float64)
    err = np.abs(rd - gd)
    tol = REL_DIST * np.abs(rd) + 1e-30
    assert np.all(err <= tol), f"distance error {err.max()} (relative {np.max(err / np.maximum(np.abs(rd), 1e-30))})"
    assert len(excused) <= max(max_excused_frac * n, 0) or len(excused) == 0 or len(excused) / n < max_excused_frac, \
        f"{len(excused)} of {n} queries needed the tie exemption"
    assert allow_excused or len(excused) == 0, f"queries {sorted(excused)[:8]} needed a tie exemption"
    assert stats["hits"] == int(ref["hit"].sum()) and stats["misses"] == n - int(ref["hit"].sum())
    return dict(ref=ref, excused=len(excused), hit_rate=float(ref["hit"].mean()))
