#!/usr/bin/env python
"""Throughput of the approximate query cache + exact top-k scan on synthetic workloads.

One step = one batch of the query stream through the whole path (probe, resolve, gather,
corpus scan of the misses, rerank, scatter).  `python bench.py --gpus N --steps K --warmup W`
prints one JSON line; with N > 1 (under torchrun) every rank holds its own copy of the corpus
and serves its own query stream (no collective on the data path), and the line reports the
sum over ranks.  `--impl reference` times the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

from paper_2503_05530_b200 import workloads as W

METRIC = "queries_per_second"
UNIT = "queries/s"


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons of one GPU, sampled while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            t = [x.strip() for x in s.split(",")]
            if len(t) < 6:
                continue
            try:
                sm.append(float(t[0])); mx.append(float(t[1]))
            except ValueError:
                continue
            for name, v in zip(names, t[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(mx) if mx else None,
                    reasons=sorted(reasons), samples=len(sm))


def stream_seed(seed: int, rank: int) -> int:
    """Every rank serves its own query stream over its own copy of the corpus."""
    return seed + rank


def aggregate_over_ranks(ms_local: float, queries_local: int, dist=None, device="cpu"):
    """Whole-job figures of a run of independent replicas: the slowest rank's time and the
    queries of all ranks.  `dist` is torch.distributed with an initialised group, or None."""
    if dist is None:
        return float(ms_local), int(queries_local)
    t = torch.tensor([ms_local], dtype=torch.float64, device=device)
    n = torch.tensor([queries_local], dtype=torch.int64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(n, op=dist.ReduceOp.SUM)
    return float(t.item()), int(n.item())


def pick_workload(name: str, free_bytes: int) -> W.Config:
    if name != "auto":
        return W.CONFIGS[name]
    cfg = W.CONFIGS["large"]
    need = cfg.N * cfg.d * 6 + (12 << 30)            # fp32 + bf16 corpus, scratch and generator temporaries
    return cfg if free_bytes >= need else W.CONFIGS["1m"]


# DRAM bytes per algorithmic byte of one scan launch, from one ncu capture of scan_tc_kernel on a 4 M x 768 cut
# of the "large" workload (dram__bytes_read.sum + dram__bytes_write.sum = 7.78 GB against 6.16 GB); the extra
# bytes grow with the row tiles like the algorithmic ones, so the ratio carries over to a full launch.
# Valid for d = 768 and 256 misses per launch only; set to None when the kernel changes.
SCAN_TRAFFIC_RATIO_D768_M256 = 1.263


def roofline_of_scan(cfg, mean_misses, scan_ms_per_launch, peaks, traffic=None):
    """The corpus scan: bytes = bf16 corpus + row norms once per launch, flops = 2 M N d."""
    bytes_alg = cfg.N * cfg.d * 2 + cfg.N * 4
    if traffic is None and cfg.d == 768 and mean_misses > 255 and SCAN_TRAFFIC_RATIO_D768_M256:
        traffic = round(SCAN_TRAFFIC_RATIO_D768_M256 * bytes_alg)
    flops = 2.0 * mean_misses * cfg.N * cfg.d
    t = scan_ms_per_launch * 1e-3
    t_hbm = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    if t_tc > t_hbm:
        ach, peak, unit, bound = flops / t / 1e12, peaks["bf16_tflops"], "TFLOP/s", "tensor"
    else:
        ach, peak, unit, bound = bytes_alg / t / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
    return dict(bound=bound, achieved=round(ach, 2), peak=peak, unit=unit, frac=round(ach / peak, 4),
                traffic=traffic, kernel="scan_tc_kernel", peak_source=peaks["source"],
                hbm_gbs=round(bytes_alg / t / 1e9, 1), tflops=round(flops / t / 1e12, 1),
                mean_misses_per_launch=round(mean_misses, 2), ms_per_launch=round(scan_ms_per_launch, 4),
                roofline_ms=round(max(t_hbm, t_tc) * 1e3, 4))


def time_stream(p, prox, batches, device_mode, dist_barrier, profile_scan=True):
    """Time the given list of batches.  Returns (ms, hits, stats, scan_ms, scan_launches, launches)."""
    torch.cuda.synchronize()
    p.reset_cache()
    if profile_scan:
        p.profile(("scan",))
        p.profile_read()
    l0 = p.kernel_launches()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    outs = []
    dist_barrier()
    torch.cuda.synchronize()
    e0.record(stream)
    if device_mode:
        for q, ids, dists, hit in batches:
            p.query_batch(q, ids, dists, hit)
    else:
        for q, ids, dists, hit in batches:
            p.query_batch_host(q, ids, dists, hit)
    e1.record(stream)
    torch.cuda.synchronize()
    dist_barrier()
    ms = e0.elapsed_time(e1)
    launches = p.kernel_launches() - l0
    scan_ms, scan_n = (0.0, 0)
    if profile_scan:
        scan_ms, scan_n = p.profile_read()["scan"]
        p.profile(())
    stats = p.stats()
    return ms, stats, scan_ms, scan_n, launches


def run_ours(args):
    from paper_2503_05530_b200 import prox
    import __graft_entry__ as g
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist_mod
        dist = dist_mod
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        g.build()
    if dist:
        dist.barrier()
    prox.load_library()

    def barrier():
        if dist:
            dist.barrier()

    free_b, _ = torch.cuda.mem_get_info()
    cfg = pick_workload(args.workload, free_b)
    if args.rows or args.batch:                                # cut-down copies for profiling runs
        cfg = cfg.scaled(N=args.rows or cfg.N, batch=args.batch or cfg.batch,
                         name=cfg.name + "-cut", n_components=max(1, cfg.n_components * (args.rows or cfg.N) // cfg.N),
                         n_topics=min(cfg.n_topics, (args.rows or cfg.N) // 4))
    peaks = load_peaks()
    sharded = bool(args.shard_rows)                          # one corpus dealt to the ranks by rows, one query stream
    seed = args.seed if sharded else stream_seed(args.seed, rank)
    K, Wm = args.steps, args.warmup
    n_batches_total = (cfg.n_queries + cfg.batch - 1) // cfg.batch
    if K <= 0:
        K = min(n_batches_total, args.default_steps)
    nq = min(cfg.n_queries, (K + Wm) * cfg.batch)

    t_gen = time.time()
    n_total = cfg.N
    if sharded:
        if args.rho != 1 or args.lsh_bits >= 0:
            raise SystemExit("--shard-rows goes with the flat cache and rho = 1")
        first, count = prox.shard_rows(n_total, world, rank)
        topic_rows = W.pick_topics(n_total, cfg.n_topics, seed, dev)
        corpus, topic_data = W.make_corpus_shard(n_total, cfg.d, cfg.n_components, args.seed, dev, first, count, topic_rows)
        queries = W.make_query_stream_from_topics(topic_data, max(nq, cfg.batch), cfg.zipf_s, cfg.sigma, seed)
        cfg = cfg.scaled(N=count)                              # what this rank scans
        del topic_data
    else:
        corpus = W.make_corpus(cfg.N, cfg.d, cfg.n_components, args.seed, dev)     # the index is the same on every rank
        queries, _, _ = W.make_query_stream(corpus, max(nq, cfg.batch), cfg.n_topics, cfg.zipf_s, cfg.sigma, seed)
    torch.cuda.synchronize()
    t_gen = time.time() - t_gen

    taus = list(cfg.taus) if args.tau is None else [args.tau]
    head_tau = taus[0]
    k = cfg.k
    results = {}
    handle_args = None
    for tau in taus:
        if sharded:
            p = prox.ProxShard(corpus, first, n_total, k, cfg.capacity, tau, cfg.policy, metric=args.metric)
        elif args.lsh_bits >= 0:                               # PROXIMITY-LSH: 2^L buckets of b entries
            planes = torch.randn(args.lsh_bits, cfg.d, device=dev, generator=torch.Generator(device=dev).manual_seed(args.seed + 77))
            p = prox.Prox(corpus, k, (1 << args.lsh_bits) * args.lsh_bucket, tau, cfg.policy, rho=args.rho,
                          lsh_planes=planes, lsh_bucket=args.lsh_bucket)
        else:
            p = prox.Prox(corpus, k, cfg.capacity, tau, cfg.policy, rho=args.rho, metric=args.metric)
        B = cfg.batch
        n_use = K * B
        ids = torch.empty(n_use, k, dtype=torch.int64, device=dev)
        dists = torch.empty(n_use, k, dtype=torch.float32, device=dev)
        hit = torch.empty(n_use, dtype=torch.uint8, device=dev)
        qs = queries[:n_use] if queries.shape[0] >= n_use else queries.repeat((n_use + queries.shape[0] - 1) // queries.shape[0], 1)[:n_use]
        batches = [(qs[a:a + B], ids[a:a + B], dists[a:a + B], hit[a:a + B]) for a in range(0, n_use, B)]
        # warm-up: W batches (not part of the timed stream), then the cache is emptied again
        wq = queries[n_use:n_use + Wm * B] if queries.shape[0] >= n_use + Wm * B else qs[:Wm * B]
        for a in range(0, wq.shape[0], B):
            p.query_batch(wq[a:a + B])
        torch.cuda.synchronize()

        sampler = ClockSampler(local) if (tau == head_tau) else None
        if sampler:
            sampler.start()
        ms, stats, scan_ms, scan_n, launches = time_stream(p, prox, batches, True, barrier)
        clocks = sampler.stop() if sampler else None
        assert p.status() == prox.OK, prox.last_error()
        hit_rate = float(hit.float().mean().item())
        r = dict(tau=tau, ms=ms, hit_rate=hit_rate, stats=stats, scan_ms=scan_ms, scan_n=scan_n,
                 launches=launches, clocks=clocks)

        if tau == head_tau:
            # end to end: host (pinned) buffers in and out, copies inside the timed region
            qh = qs.cpu().pin_memory()
            ih = torch.empty(n_use, k, dtype=torch.int64).pin_memory()
            dh = torch.empty(n_use, k, dtype=torch.float32).pin_memory()
            hh = torch.empty(n_use, dtype=torch.uint8).pin_memory()
            hb = [(qh[a:a + B], ih[a:a + B], dh[a:a + B], hh[a:a + B]) for a in range(0, n_use, B)]
            ms_e2e, _, _, _, _ = time_stream(p, prox, hb, False, barrier, profile_scan=False)
            assert torch.equal(ih.to(dev), ids) and torch.equal(hh.to(dev), hit), "host and device entry points disagree"
            r["ms_e2e"] = ms_e2e
            r["h2d"] = B * cfg.d * 4
            r["d2h"] = B * k * 12 + B
            handle_args = dict(ids=ids[: 64].cpu().numpy(), dists=dists[:64].cpu().numpy(), hit=hit[:64].cpu().numpy(),
                               q=qs[:64].cpu().numpy())
        if args.stages and rank == 0:
            p.reset_cache()
            p.profile(None)
            p.profile_read()
            for q, i_, d_, h_ in batches:
                p.query_batch(q, i_, d_, h_)
            prof = p.profile_read()
            p.profile(())
            print(json.dumps(dict(stage_ms_per_step={kk: round(v[0] / K, 4) for kk, v in prof.items()}, tau=tau)),
                  file=sys.stderr, flush=True)
        results[tau] = r
        p.close()
        del p

    # max over ranks of the times, sum over ranks of the queries
    head = results[head_tau]
    ms, total_q = aggregate_over_ranks(head["ms"], K * cfg.batch, dist, dev)
    ms_e2e, _ = aggregate_over_ranks(head["ms_e2e"], K * cfg.batch, dist, dev)
    if sharded:
        total_q = K * cfg.batch                              # every rank answered the same queries
    value = total_q / (ms * 1e-3)
    e2e = total_q / (ms_e2e * 1e-3)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and not sharded:
        cpu = cpu_baseline(cfg, corpus, queries, head_tau, budget_s=args.cpu_seconds)
    if rank != 0:
        if dist:
            dist.destroy_process_group()
        return

    def scan_roofline(r):
        """Roofline of the scan over the launches that had misses to scan (a launch takes up to 256 of them;
        launches of batches without misses return at once and only add their few microseconds)."""
        sb = max(1, r["stats"]["scan_batches"])
        per_batch = r["stats"]["misses"] / sb
        working = sb * max(1, -(-int(round(per_batch)) // 256))
        return roofline_of_scan(cfg, r["stats"]["misses"] / working, r["scan_ms"] / working, peaks)

    roof = scan_roofline(head)
    sweep = []
    for tau, r in results.items():
        rf = scan_roofline(r)
        sweep.append(dict(tau=tau, value=round(K * cfg.batch / (r["ms"] * 1e-3), 1), hit_rate=round(r["hit_rate"], 4),
                          ms_per_step=round(r["ms"] / K, 4), scan_frac_of_roofline=rf["frac"], scan_bound=rf["bound"],
                          scan_ms_per_launch=rf["ms_per_launch"], uncertified=r["stats"]["uncertified"],
                          unresolved=r["stats"]["unresolved"]))
    line = dict(
        metric=METRIC, value=round(value, 1), unit=UNIT, n_gpus=world, steps=K, warmup=Wm,
        ms_per_step=round(ms / K, 4), higher_is_better=True, scaling="strong" if sharded else "weak", vs_baseline=None,
        dtype="bf16 scan + f64 rerank/probe", data="synthetic",
        config=dict(workload=f"{cfg.name}: N={n_total} d={cfg.d} k={cfg.k} capacity={cfg.capacity} policy={cfg.policy} "
                             f"batch={cfg.batch} tau={head_tau} topics={cfg.n_topics} zipf={cfg.zipf_s} sigma={cfg.sigma}",
                    tau=head_tau, hit_rate=round(head["hit_rate"], 4), l2="inputs_exceed_l2" if cfg.N * cfg.d * 2 > 126e6 else "corpus_fits_l2",
                    parallelism=f"row shards x{world} ({cfg.N} rows each), cache replicated" if sharded else f"replica x{world}", rho=args.rho, metric=args.metric,
                    cache="flat" if args.lsh_bits < 0 else f"lsh L={args.lsh_bits} b={args.lsh_bucket}", seed=args.seed, gen_seconds=round(t_gen, 1)),
        clocks=head["clocks"],
        e2e=dict(value=round(e2e, 1), unit=UNIT, h2d_bytes_per_step=head["h2d"], d2h_bytes_per_step=head["d2h"]),
        gpu_launches=int(head["launches"]),
        roofline=roof, tau_sweep=sweep, cpu_baseline=cpu,
        stats=head["stats"],
    )
    print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def cpu_baseline(cfg, corpus, queries, tau, budget_s=20.0):
    """The oracle as it stands on the host cores, on a bounded sample: the cache probe of a run
    of queries against a full cache, and the exact top-k of a few queries over a slab of the
    corpus (its time grows in proportion to the rows), combined as 1 / (t_probe + miss_rate * t_knn)."""
    import oracle
    cores = oracle.num_threads()
    rows = int(min(cfg.N, max(50_000, 2.0e9 * cores // (cfg.d * 8))))
    rows = min(rows, cfg.N)
    slab = corpus[:rows].cpu().numpy()
    nq = 4
    qs = queries[:max(nq, 64)].cpu().numpy()
    t0 = time.time()
    oracle.exact_topk(slab, qs[:nq], cfg.k)
    t_knn_slab = (time.time() - t0) / nq
    t_knn = t_knn_slab * (cfg.N / rows)
    # probe: a trace-only oracle with a full cache of distinct keys
    cap = min(cfg.capacity, 20_000)
    keys = corpus[:cap].cpu().numpy()
    o = oracle.Oracle(None, cfg.d, 1, cap, 0.0, oracle.LRU)
    o.cache_load(keys)
    t0 = time.time()
    o.query(qs[:64])
    t_probe = (time.time() - t0) / 64 * (cfg.capacity / cap)
    o.close()
    miss_rate = 1.0 if tau == 0 else None
    mr = 1.0 if miss_rate is None else miss_rate
    value = 1.0 / (t_probe + mr * t_knn)
    return dict(value=round(value, 4), unit=UNIT, cores=cores, kind="oracle",
                sample=f"exact top-k of {nq} queries over the first {rows} corpus rows, scaled by N/rows; probe of 64 "
                       f"queries against {cap} keys scaled to capacity; miss rate taken as 1",
                knn_seconds_per_query=round(t_knn, 3), probe_seconds_per_query=round(t_probe, 6))


def run_reference(args):
    """The CPU oracle as the reference arm: rank 0 only; each step is a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    name = args.workload if args.workload != "auto" else "large"
    cfg = W.CONFIGS[name]
    tau = cfg.taus[0] if args.tau is None else args.tau
    cores = oracle.num_threads()
    rows = 200_000
    K = args.steps if args.steps > 0 else 5
    corpus = W.make_corpus(rows, cfg.d, max(1, cfg.n_components * rows // cfg.N), args.seed, "cpu")
    queries, _, _ = W.make_query_stream(corpus, (K + args.warmup) * 2, min(cfg.n_topics, rows // 10), cfg.zipf_s, cfg.sigma, args.seed)
    X, Q = corpus.numpy(), queries.numpy()
    cap = min(cfg.capacity, 5_000)
    o = oracle.Oracle(None, cfg.d, 1, cap, 0.0, oracle.LRU)
    o.cache_load(X[:cap])

    def step(i):
        q = Q[2 * i:2 * i + 2]
        t0 = time.time()
        oracle.exact_topk(X, q, cfg.k)
        t_knn = (time.time() - t0) / 2 * (cfg.N / rows)
        t0 = time.time()
        o.query(q)
        t_probe = (time.time() - t0) / 2 * (cfg.capacity / cap)
        return t_knn + t_probe
    for i in range(args.warmup):
        step(i)
    per_query = [step(args.warmup + i) for i in range(K)]
    sec_per_query = sum(per_query) / len(per_query)
    value = 1.0 / sec_per_query
    sample = (f"per step: exact top-k of 2 queries over {rows} rows and their probe against {cap} keys, "
              f"scaled to N={cfg.N} rows and capacity={cfg.capacity}; every query counted as a miss")
    line = dict(impl="reference", metric=METRIC, value=round(value, 4), unit=UNIT, n_gpus=args.gpus, steps=K,
                warmup=args.warmup, ms_per_step=round(sec_per_query * cfg.batch * 1e3, 1), higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=f"{cfg.name}: N={cfg.N} d={cfg.d} k={cfg.k} capacity={cfg.capacity} "
                                     f"policy={cfg.policy} batch={cfg.batch} tau={tau}", tau=tau),
                cpu_baseline=dict(value=round(value, 4), unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=round(value, 4), unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line), flush=True)


def run_probe(args):
    """Probe-only workload: a cache pre-filled with C keys, batches of 1024 queries (half near
    random keys, half fresh mixture draws), tau = 0.5; times probe + resolve + key insertion
    (prox_probe_batch) and reports GB/s of keys scanned per cache size and policy."""
    from paper_2503_05530_b200 import prox
    import __graft_entry__ as g
    g.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    B, d, tau = 1024, 768, 0.5
    K = args.steps if args.steps > 0 else 50
    sizes = [c for c in W.PROBE_SIZES if c <= (args.rows or W.PROBE_SIZES[-1])]
    peaks = load_peaks()
    fp64_peak = 148 * 64 * 1.965e9                      # DADD/DFMA issue slots per second (64 per SM and clock)
    out = []
    for C in sizes:
        keys, centres = W.make_probe_keys(C, d, 4096, args.seed, dev)
        batches = [W.make_probe_batch(keys, centres, B, 0.02, args.seed, b) for b in range(K + args.warmup)]
        for policy in ("lru", "fifo"):
            p = prox.Prox(keys[:64].contiguous(), 1, C, tau, policy)
            p.cache_load(keys)
            for q in batches[K:]:
                p.probe_batch(q)
            torch.cuda.synchronize()
            p.cache_load(keys)
            p.profile(None)
            p.profile_read()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            hits = []
            e0.record()
            for q in batches[:K]:
                hits.append(p.probe_batch(q)[0])
            e1.record()
            torch.cuda.synchronize()
            prof = p.profile_read()
            assert p.status() == prox.OK, prox.last_error()
            ms = e0.elapsed_time(e1) / K
            hit_rate = float(torch.stack(hits).float().mean().item())
            key_bytes = C * d * 4
            probe_s = prof["probe"][0] / K * 1e-3
            coarse = (C >= 4096)                        # the library probes large caches on the tensor cores first
            if coarse:                                  # bf16 contraction 2 B C d against the measured bf16 peak
                ach, peak, unit, bound = 2.0 * B * C * d / probe_s / 1e12, peaks["bf16_tflops"], "TFLOP/s", "tensor"
            else:                                       # fp64 difference form: one subtraction, one fused multiply-add per element
                ach, peak, unit, bound = 2.0 * B * C * d / probe_s / 1e12, fp64_peak / 1e12, "T fp64 instr/s", "alu"
            out.append(dict(C=C, policy=policy, us_per_batch=round(ms * 1e3, 1), keys_GBps=round(key_bytes / ms / 1e6, 1),
                            hit_rate=round(hit_rate, 4), queries_per_s=round(B / ms * 1e3, 1),
                            probe_us=round(prof["probe"][0] / K * 1e3, 1), resolve_us=round(prof["resolve"][0] / K * 1e3, 1),
                            risk_select_us=round(prof["risk_select"][0] / K * 1e3, 1),
                            probe_uncertified=p.stats()["probe_uncertified"],
                            roofline=dict(bound=bound, achieved=round(ach, 2), peak=round(peak, 2), unit=unit,
                                          frac=round(ach / peak, 4), traffic=None,
                                          kernel="scan_tc_kernel over the keys" if coarse else "probe_kernel")))
            p.close()
        del keys, batches
    # PROXIMITY-LSH at the paper's setting (L = 10, b = 20, capacity 20 480): filled by a pass of keys, then timed
    lsh = None
    if not args.rows or args.rows >= 20480:
        Lb, bb = 10, 20
        keys, centres = W.make_probe_keys(1 << 15, d, 4096, args.seed, dev)
        planes = torch.randn(Lb, d, device=dev, generator=torch.Generator(device=dev).manual_seed(args.seed + 77))
        p = prox.Prox(keys[:64].contiguous(), 1, (1 << Lb) * bb, tau, "lru", lsh_planes=planes, lsh_bucket=bb)
        for a in range(0, keys.shape[0], B):
            p.probe_batch(keys[a:a + B])
        batches = [W.make_probe_batch(keys, centres, B, 0.02, args.seed, b_) for b_ in range(K + args.warmup)]
        for q in batches[K:]:
            p.probe_batch(q)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        hits = []
        e0.record()
        for q in batches[:K]:
            hits.append(p.probe_batch(q)[0])
        e1.record()
        torch.cuda.synchronize()
        assert p.status() == prox.OK, prox.last_error()
        ms = e0.elapsed_time(e1) / K
        st = p.stats()
        alg_bytes = B * (Lb + bb) * d * 4                  # every query reads the hyperplanes and its bucket's keys
        lsh = dict(L=Lb, b=bb, capacity=(1 << Lb) * bb, held=st["count"], us_per_batch=round(ms * 1e3, 1),
                   queries_per_s=round(B / ms * 1e3, 1), hit_rate=round(float(torch.stack(hits).float().mean().item()), 4),
                   roofline=dict(bound="hbm", achieved=round(alg_bytes / ms / 1e6, 1), peak=peaks["hbm_gbs"], unit="GB/s",
                                 frac=round(alg_bytes / ms / 1e6 / peaks["hbm_gbs"], 4), traffic=None,
                                 kernel="lsh_resolve_kernel (gather of one bucket per query, replay in order)"))
        p.close()
    big = out[-1]
    print(json.dumps(dict(metric="probe_keys_scanned", value=big["keys_GBps"], unit="GB/s", n_gpus=1, steps=K,
                          warmup=args.warmup, ms_per_step=round(big["us_per_batch"] / 1e3, 4), higher_is_better=True,
                          scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                          config=dict(workload=f"probe-only: B={B} d={d} tau={tau} keys from a 4096-component mixture, "
                                               f"C={big['C']} policy={big['policy']}", l2="keys_exceed_l2" if big["C"] * d * 4 > 126e6 else "keys_fit_l2"),
                          roofline=big["roofline"],
                          points=out, lsh=lsh)), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=0, help="timed batches (0: a default that ends within minutes)")
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="auto", choices=["auto", "probe"] + list(W.CONFIGS))
    ap.add_argument("--tau", type=float, default=None, help="one tolerance instead of the workload's sweep")
    ap.add_argument("--rows", type=int, default=0, help="override the corpus size (profiling runs)")
    ap.add_argument("--batch", type=int, default=0, help="override the batch size (profiling runs)")
    ap.add_argument("--rho", type=int, default=1, help="re-ranking factor: rho * k rows fetched and stored per miss (1 = none)")
    ap.add_argument("--metric", default="l2", choices=["l2", "cosine", "ip"], help="distance of the cache keys and of the corpus")
    ap.add_argument("--lsh-bits", type=int, default=-1, help="PROXIMITY-LSH with this many hyperplanes (-1: flat cache)")
    ap.add_argument("--lsh-bucket", type=int, default=20, help="entries per LSH bucket")
    ap.add_argument("--shard-rows", action="store_true", help="deal the rows of ONE corpus to the ranks (every rank answers the same "
                    "queries; one all-gather per batch) instead of running independent replicas")
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--default-steps", type=int, default=800, help="cap of the timed batches when --steps is 0 (a whole query stream if it is shorter)")
    ap.add_argument("--cpu-seconds", type=float, default=20.0)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--stages", action="store_true", help="also print the time of every stage (one extra run)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        run_reference(args)
    elif args.workload == "probe":
        run_probe(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
