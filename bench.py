#!/usr/bin/env python
"""Throughput of the approximate query cache + exact top-k scan on synthetic workloads.

One step = one batch of the query stream through the whole path (probe, resolve, gather,
corpus scan of the misses, rerank, scatter).  `python bench.py --gpus N --steps K --warmup W`
prints one JSON line.  Its headline is the 24 M x 768 workload (the 1 M x 768 one when the GPU
is too small); with no `--workload` given and one GPU the line also carries, under `workloads`,
the other published configurations (10 k x 768 one query at a time, 1 M x 768 with its five
tolerances, 100 M x 128, the probe-only cache sizes under LRU and FIFO, the LSH cache) and,
under `sustained`, the headline tolerance timed again over a few hundred batches.  With N > 1
(under torchrun) every rank holds its own copy of the corpus and serves its own query stream (no
collective on the data path), the line reports the sum over ranks, and a `shard_rows` record
times ONE corpus dealt to the ranks by rows (one all-gather per batch).  `--impl reference` times
the CPU oracle on a bounded sample instead.
"""
from __future__ import annotations

import argparse
import gc
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
DTYPE = "bf16 scan + f64 rerank/probe"


def load_peaks():
    """Measured peaks of this machine's GPUs.  `bf16_tflops` is the burst figure of a dense GEMM (the
    denominator of every tensor fraction reported here); `bf16_tflops_sustained` is the same GEMM in
    a seconds-long loop under the power cap, reported beside it."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        burst = float(p["bf16_tflops"])
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=burst,
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", burst)), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks, throttle reasons and power draw of one GPU (read only).  The sampler is started ahead of the timed region
    (the tool needs a few hundred milliseconds before its first line) and keeps the time stamp of every sample;
    `stop` reports the samples taken between `begin()` and `end()` (all of them if none was marked)."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
              "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None
        self.t0 = self.t1 = None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                                          "--format=csv,noheader,nounits", "-lms", "50"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except OSError:
            self.proc = None
        return self

    def begin(self):
        self.t0 = time.time()

    def end(self):
        self.t1 = time.time()

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append(line.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        if self.t1 is not None:                               # let a sample that was under way at the end come in
            time.sleep(0.06)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        import datetime
        rows = []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for s in self.samples:
            t = [x.strip() for x in s.split(",")]
            if len(t) < 7:
                continue
            try:
                ts = datetime.datetime.strptime(t[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                try:
                    watts = float(t[7]) if len(t) > 7 else None
                except ValueError:
                    watts = None
                rows.append((ts, float(t[1]), float(t[2]), [n for n, v in zip(names, t[3:7]) if v.lower().startswith("active")], watts))
            except ValueError:
                continue
        inside = rows
        if self.t0 is not None and self.t1 is not None:
            inside = [r for r in rows if self.t0 <= r[0] <= self.t1 + 0.05]
            if not inside and rows:                           # a region shorter than the sampling period: the nearest sample
                mid = 0.5 * (self.t0 + self.t1)
                inside = [min(rows, key=lambda r: abs(r[0] - mid))]
        sm = [r[1] for r in inside]
        reasons = sorted({n for r in inside for n in r[3]})
        watts = [r[4] for r in inside if r[4] is not None]
        return dict(sm_mhz=statistics.median(sm) if sm else None, sm_max_mhz=max(r[2] for r in inside) if inside else None,
                    reasons=reasons, samples=len(sm), power_w=round(statistics.median(watts), 1) if watts else None)


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


def workload_text(cfg, tau, n_total=None) -> str:
    """The one description of a workload that both arms print."""
    return (f"{cfg.name}: N={n_total or cfg.N} d={cfg.d} k={cfg.k} capacity={cfg.capacity} policy={cfg.policy} "
            f"batch={cfg.batch} tau={tau} topics={cfg.n_topics} zipf={cfg.zipf_s} sigma={cfg.sigma}")


def pick_workload(name: str, free_bytes: int) -> W.Config:
    if name != "auto":
        return W.CONFIGS[name]
    cfg = W.CONFIGS["large"]
    need = cfg.N * cfg.d * 6 + (12 << 30)            # fp32 + bf16 corpus, scratch and generator temporaries
    return cfg if free_bytes >= need else W.CONFIGS["1m"]


# DRAM traffic of one scan launch, from an ncu capture of scan_tc_kernel on a 1 M-row cut of the 24 M x 768 workload
# (dram__bytes_read.sum = 1.5502 GB against 1.5400 GB of bf16 rows + norms; dram__bytes_write.sum = 0.0943 GB of
# candidate appends while the thresholds of the first tiles are still open).  The bytes read grow with the row tiles
# like the algorithmic ones, the appends do not, so a full launch is taken as ratio x algorithmic + appends.  Valid
# for d = 768 and 256 misses per launch only; None once the kernel has changed since the counters were taken.
SCAN_TRAFFIC_D768_M256 = dict(read_ratio=1.0066, append_bytes=94_348_544)


def roofline_of_scan(cfg, mean_misses, scan_ms_per_launch, peaks, clocks=None, traffic=None):
    """The corpus scan: bytes = bf16 corpus + row norms once per launch, flops = 2 M N d.  The fraction is taken
    against the burst bf16 figure (or the copy bandwidth); the sustained figure stands beside it."""
    bytes_alg = cfg.N * cfg.d * 2 + cfg.N * 4
    if traffic is None and cfg.d == 768 and mean_misses > 255 and SCAN_TRAFFIC_D768_M256:
        traffic = round(SCAN_TRAFFIC_D768_M256["read_ratio"] * bytes_alg + SCAN_TRAFFIC_D768_M256["append_bytes"])
    flops = 2.0 * mean_misses * cfg.N * cfg.d
    t = max(scan_ms_per_launch, 1e-9) * 1e-3
    t_hbm = bytes_alg / (peaks["hbm_gbs"] * 1e9)
    t_tc = flops / (peaks["bf16_tflops"] * 1e12)
    more = dict()
    if t_tc > t_hbm:
        ach, peak, unit, bound = flops / t / 1e12, peaks["bf16_tflops"], "TFLOP/s", "tensor"
        more["frac_of_sustained_peak"] = round(ach / peaks["bf16_tflops_sustained"], 4)
        more["peak_sustained"] = peaks["bf16_tflops_sustained"]
    else:
        ach, peak, unit, bound = bytes_alg / t / 1e9, peaks["hbm_gbs"], "GB/s", "hbm"
    out = dict(bound=bound, achieved=round(ach, 2), peak=peak, unit=unit, frac=round(ach / peak, 4),
               traffic=traffic, kernel="scan_tc_multi_kernel" if (cfg.d <= 128 and cfg.batch > 256) else "scan_tc_kernel",
               peak_source=peaks["source"],
               peak_kind="burst bf16 GEMM" if bound == "tensor" else "copy bandwidth", **more,
               hbm_gbs=round(bytes_alg / t / 1e9, 1), tflops=round(flops / t / 1e12, 1),
               mean_misses_per_launch=round(mean_misses, 2), ms_per_launch=round(scan_ms_per_launch, 4),
               roofline_ms=round(max(t_hbm, t_tc) * 1e3, 4))
    if clocks and clocks.get("sm_mhz"):
        out["ms_x_sm_ghz"] = round(scan_ms_per_launch * clocks["sm_mhz"] / 1e3, 3)   # million SM cycles per launch
    return out


def time_stream(p, batches, device_mode, dist_barrier, profile_scan=True):
    """Time the given list of batches.  Returns (ms, stats, scan_ms, scan_launches, launches)."""
    torch.cuda.synchronize()
    p.reset_cache()
    if profile_scan:
        p.profile(("scan",))
        p.profile_read()
    l0 = p.kernel_launches()
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
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


def time_stream_replayed(p, batches, dist_barrier):
    """The same batches through one recorded batch call (prox_record_batch / prox_replay_batch): every step
    copies its queries into the recording's fixed buffer (device to device, inside the timed region) and
    replays.  Returns (ms, stats, hit flags of the last batch)."""
    q0, i0, d0, h0 = batches[0]
    dev = q0.device
    qb, ib, db, hb = torch.empty_like(q0), torch.empty_like(i0), torch.empty_like(d0), torch.empty_like(h0)
    torch.cuda.synchronize()
    p.reset_cache()
    side = torch.cuda.Stream(device=dev)             # stream capture needs a stream other than the legacy default one
    side.wait_stream(torch.cuda.current_stream(dev))
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(side):
        rec = p.record_batch(qb, ib, db, hb, stream=side)
        dist_barrier()
        side.synchronize()
        e0.record(side)
        for q, _, _, _ in batches:
            qb.copy_(q, non_blocking=True)
            rec.replay(stream=side)
        e1.record(side)
        side.synchronize()
    dist_barrier()
    ms = e0.elapsed_time(e1)
    stats = p.stats()
    rec.close()
    return ms, stats, hb


def scan_roofline(cfg, r, peaks):
    """Roofline of the scan over the launches that had misses to scan (a launch takes up to 256 of them;
    launches of batches without misses return at once and only add their few microseconds)."""
    sb = max(1, r["stats"]["scan_batches"])
    per_batch = r["stats"]["misses"] / sb
    working = sb * max(1, -(-int(round(per_batch)) // 256))
    return roofline_of_scan(cfg, r["stats"]["misses"] / working, r["scan_ms"] / working, peaks, r.get("clocks"))


def run_streams(prox, cfg, queries, taus, K, Wm, dev, local, barrier, make_handle, peaks, e2e=True, stages=False,
                sustained_steps=0, replay=False):
    """The query stream of a workload through one handle per tolerance: W untimed batches, then K
    timed ones from an empty cache (CUDA events on the launching stream); for the first tolerance
    also the same batches through the host-buffer entry point, and the long run."""
    results, extra = {}, {}
    head_tau = taus[0]
    k, B = cfg.k, cfg.batch
    n_use = K * B
    for tau in taus:
        p = make_handle(tau)
        ids = torch.empty(n_use, k, dtype=torch.int64, device=dev)
        dists = torch.empty(n_use, k, dtype=torch.float32, device=dev)
        hit = torch.empty(n_use, dtype=torch.uint8, device=dev)
        qs = queries[:n_use] if queries.shape[0] >= n_use else queries.repeat((n_use + queries.shape[0] - 1) // queries.shape[0], 1)[:n_use]
        batches = [(qs[a:a + B], ids[a:a + B], dists[a:a + B], hit[a:a + B]) for a in range(0, n_use, B)]
        wq = queries[n_use:n_use + Wm * B] if queries.shape[0] >= n_use + Wm * B else qs[:Wm * B]
        sampler = ClockSampler(local).start()
        for a in range(0, wq.shape[0], B):
            p.query_batch(wq[a:a + B])
        torch.cuda.synchronize()
        sampler.begin()
        ms, stats, scan_ms, scan_n, launches = time_stream(p, batches, True, barrier)
        sampler.end()
        clocks = sampler.stop()
        assert p.status() == prox.OK, prox.last_error()
        r = dict(tau=tau, ms=ms, hit_rate=float(hit.float().mean().item()), stats=stats, scan_ms=scan_ms, scan_n=scan_n,
                 launches=launches, clocks=clocks)
        if tau == head_tau and e2e:
            # end to end: host (pinned) buffers in and out, copies inside the timed region
            qh = qs.cpu().pin_memory()
            ih = torch.empty(n_use, k, dtype=torch.int64).pin_memory()
            dh = torch.empty(n_use, k, dtype=torch.float32).pin_memory()
            hh = torch.empty(n_use, dtype=torch.uint8).pin_memory()
            hb = [(qh[a:a + B], ih[a:a + B], dh[a:a + B], hh[a:a + B]) for a in range(0, n_use, B)]
            ms_e2e, _, _, _, _ = time_stream(p, hb, False, barrier, profile_scan=False)
            assert torch.equal(ih.to(dev), ids) and torch.equal(hh.to(dev), hit), "host and device entry points disagree"
            r["ms_e2e"], r["h2d"], r["d2h"] = ms_e2e, B * cfg.d * 4, B * k * 12 + B
        if tau == head_tau and sustained_steps > 0:
            # the same tolerance over a long run: seconds under the power cap, the whole stream if it is shorter
            n_long = min(sustained_steps, queries.shape[0] // B) * B
            ql = queries[:n_long]
            il = torch.empty(B, k, dtype=torch.int64, device=dev)
            dl = torch.empty(B, k, dtype=torch.float32, device=dev)
            hl = torch.empty(n_long, dtype=torch.uint8, device=dev)
            lb = [(ql[a:a + B], il, dl, hl[a:a + B]) for a in range(0, n_long, B)]
            sampler = ClockSampler(local).start()
            sampler.begin()
            ms_l, st_l, scan_l, _, _ = time_stream(p, lb, True, barrier)
            sampler.end()
            ck = sampler.stop()
            rf = scan_roofline(cfg, dict(stats=st_l, scan_ms=scan_l, clocks=ck), peaks)
            extra["sustained"] = dict(tau=tau, steps=n_long // B, value=round(n_long / (ms_l * 1e-3), 1), unit=UNIT,
                                      ms_per_step=round(ms_l / (n_long // B), 4), hit_rate=round(float(hl.float().mean().item()), 4),
                                      scan_ms_per_launch=rf["ms_per_launch"], scan_bound=rf["bound"], scan_frac=rf["frac"],
                                      scan_frac_of_sustained_peak=rf.get("frac_of_sustained_peak"),
                                      ms_x_sm_ghz=rf.get("ms_x_sm_ghz"), clocks=ck)
        if tau == head_tau and replay:
            # launch-bound shapes: the batch call recorded once and replayed (same batches, same counters)
            ms_r, st_r, _ = time_stream_replayed(p, batches, barrier)
            same = all(st_r[kk] == stats[kk] for kk in ("queries", "hits", "misses", "evictions", "intra_batch_hits"))
            assert same, "the replayed stream and the plain stream disagree"
            r["ms_replayed"] = ms_r
        if stages:
            p.reset_cache()
            p.profile(None)
            p.profile_read()
            for q, i_, d_, h_ in batches:
                p.query_batch(q, i_, d_, h_)
            prof = p.profile_read()
            p.profile(())
            r["stage_ms_per_step"] = {kk: round(v[0] / K, 4) for kk, v in prof.items()}
            print(json.dumps(dict(workload=cfg.name, stage_ms_per_step=r["stage_ms_per_step"], tau=tau)), file=sys.stderr, flush=True)
        results[tau] = r
        p.close()
        del p
    return results, extra


def sweep_rows(cfg, results, K, peaks):
    out = []
    for tau, r in results.items():
        rf = scan_roofline(cfg, r, peaks)
        row = dict(tau=tau, value=round(K * cfg.batch / (r["ms"] * 1e-3), 1), hit_rate=round(r["hit_rate"], 4),
                   ms_per_step=round(r["ms"] / K, 4), scan_frac_of_roofline=rf["frac"], scan_bound=rf["bound"],
                   scan_ms_per_launch=rf["ms_per_launch"], uncertified=r["stats"]["uncertified"],
                   unresolved=r["stats"]["unresolved"])
        if "frac_of_sustained_peak" in rf:
            row["scan_frac_of_sustained_peak"] = rf["frac_of_sustained_peak"]
        if "stage_ms_per_step" in r:
            row["stage_ms_per_step"] = r["stage_ms_per_step"]
        out.append(row)
    return out


def run_extra_stream_workload(prox, name, args, dev, local, peaks, K, stages=True):
    """One of the other published configurations, reported under `workloads` (own clocks record)."""
    cfg = W.CONFIGS[name]
    free_b, _ = torch.cuda.mem_get_info()
    need = cfg.N * cfg.d * 6 + (10 << 30)
    if free_b < need:
        return dict(skipped=f"needs {need >> 30} GB of free device memory, {free_b >> 30} GB free")
    Wm = 3
    taus = list(cfg.taus)
    K = min(K, (cfg.n_queries + cfg.batch - 1) // cfg.batch)
    nq = min(cfg.n_queries, (K + Wm) * cfg.batch)
    t0 = time.time()
    corpus = W.make_corpus(cfg.N, cfg.d, cfg.n_components, args.seed, dev)
    queries, _, _ = W.make_query_stream(corpus, max(nq, cfg.batch), cfg.n_topics, cfg.zipf_s, cfg.sigma, args.seed)
    torch.cuda.synchronize()
    t_gen = time.time() - t0
    results, _ = run_streams(prox, cfg, queries, taus, K, Wm, dev, local, lambda: None,
                             lambda tau: prox.Prox(corpus, cfg.k, cfg.capacity, tau, cfg.policy), peaks, e2e=False, stages=stages,
                             replay=cfg.batch <= 64)
    head = results[taus[0]]
    rf = scan_roofline(cfg, head, peaks)
    out = dict(workload=workload_text(cfg, taus[0]), steps=K, warmup=Wm, value=round(K * cfg.batch / (head["ms"] * 1e-3), 1), unit=UNIT,
               ms_per_step=round(head["ms"] / K, 4), us_per_query=round(head["ms"] * 1e3 / (K * cfg.batch), 3),
               hit_rate=round(head["hit_rate"], 4), gpu_launches=int(head["launches"]), clocks=head["clocks"],
               roofline=rf, tau_sweep=sweep_rows(cfg, results, K, peaks), gen_seconds=round(t_gen, 1),
               l2="inputs_exceed_l2" if cfg.N * cfg.d * 2 > 126e6 else "corpus_fits_l2")
    if "ms_replayed" in head:
        mr = head["ms_replayed"]
        out["replayed"] = dict(value=round(K * cfg.batch / (mr * 1e-3), 1), unit=UNIT, ms_per_step=round(mr / K, 4),
                               us_per_query=round(mr * 1e3 / (K * cfg.batch), 3),
                               how="prox_record_batch once, then per step a device-to-device copy of the queries into "
                                   "the recording's buffer and prox_replay_batch; same batches, same counters")
    del corpus, queries
    gc.collect()
    torch.cuda.empty_cache()
    return out


def cpu_baseline(cfg, corpus, queries, tau, budget_s=20.0):
    """The oracle as it stands on the host cores, on a bounded sample: the exact top-k of S = 32 queries over a
    slab of the corpus (its time grows in proportion to the rows), on all cores and on one, and the cache
    probe of 64 queries against a full cache; combined as 1 / (t_probe + miss_rate * t_knn) and extrapolated."""
    import oracle
    cores = oracle.num_threads()
    S = 32
    per_row_s = cfg.d * 0.55e-9                        # about 1.8 G multiply-adds per second and core
    slab_rows = int(3.0e9 // (cfg.d * 4))              # at most 3 GB of rows leave the device
    rows = int(min(cfg.N, slab_rows, max(20_000, budget_s * 0.4 * cores / (2 * S * per_row_s))))
    rows1 = int(min(rows, max(5_000, budget_s * 0.3 / (S * per_row_s))))
    slab = corpus[:rows].cpu().numpy()
    qs = queries[:2 * S].cpu().numpy()
    oracle.exact_topk(slab[:1000], qs[:1], min(cfg.k, 1000))            # page the library in
    t0 = time.time()
    oracle.exact_topk(slab, qs[:2 * S], cfg.k)
    t_knn = (time.time() - t0) / (2 * S) * (cfg.N / rows)
    oracle.set_threads(1)
    t0 = time.time()
    oracle.exact_topk(slab[:rows1], qs[:S], min(cfg.k, rows1))
    t_knn1 = (time.time() - t0) / S * (cfg.N / rows1)
    oracle.set_threads(cores)
    # probe: a trace-only oracle with a full cache of distinct keys (one core: the replay is sequential)
    cap = min(cfg.capacity, 20_000)
    keys = corpus[:cap].cpu().numpy()
    o = oracle.Oracle(None, cfg.d, 1, cap, 0.0, oracle.LRU)
    o.cache_load(keys)
    t0 = time.time()
    o.query(qs[:64])
    t_probe = (time.time() - t0) / 64 * (cfg.capacity / cap)
    o.close()
    value = 1.0 / (t_probe + t_knn)
    value1 = 1.0 / (t_probe + t_knn1)
    return dict(value=round(value, 4), unit=UNIT, cores=cores, kind="oracle",
                sample=f"extrapolated from {2 * S} queries: exact top-k of {2 * S} queries over the first {rows} corpus rows on {cores} "
                       f"cores (and of {S} queries over the first {rows1} rows on one core), scaled by N/rows; probe of 64 queries against "
                       f"{cap} keys on one core, scaled to capacity; every query counted as a miss (tau = {tau})",
                single_thread_value=round(value1, 5), knn_seconds_per_query=round(t_knn, 3),
                knn_seconds_per_query_single_thread=round(t_knn1, 2), probe_seconds_per_query=round(t_probe, 6))


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
    base_cfg = cfg
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
    plain = (not sharded and not args.rows and not args.batch and args.tau is None and args.rho == 1 and
             args.metric == "l2" and args.lsh_bits < 0 and not args.no_extras)
    extras_on = plain and args.workload == "auto" and world == 1
    long_steps = args.sustained_steps if (extras_on or args.sustained) else 0
    nq = min(cfg.n_queries, max((K + Wm) * cfg.batch, long_steps * cfg.batch))

    t_gen = time.time()
    n_total = cfg.N
    first = 0
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

    def make_handle(tau):
        if sharded:
            return prox.ProxShard(corpus, first, n_total, cfg.k, cfg.capacity, tau, cfg.policy, metric=args.metric)
        if args.lsh_bits >= 0:                                 # PROXIMITY-LSH: 2^L buckets of b entries
            planes = torch.randn(args.lsh_bits, cfg.d, device=dev, generator=torch.Generator(device=dev).manual_seed(args.seed + 77))
            return prox.Prox(corpus, cfg.k, (1 << args.lsh_bits) * args.lsh_bucket, tau, cfg.policy, rho=args.rho,
                             lsh_planes=planes, lsh_bucket=args.lsh_bucket)
        return prox.Prox(corpus, cfg.k, cfg.capacity, tau, cfg.policy, rho=args.rho, metric=args.metric)

    results, extra = run_streams(prox, cfg, queries, taus, K, Wm, dev, local, barrier, make_handle, peaks, e2e=True,
                                 stages=bool(args.stages) and rank == 0, sustained_steps=long_steps,
                                 replay=cfg.batch <= 64 and not sharded)

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

    line = None
    if rank == 0:
        roof = scan_roofline(cfg, head, peaks)
        line = dict(
            metric=METRIC, value=round(value, 1), unit=UNIT, n_gpus=world, steps=K, warmup=Wm,
            ms_per_step=round(ms / K, 4), higher_is_better=True, scaling="strong" if sharded else "weak", vs_baseline=None,
            dtype=DTYPE, data="synthetic",
            config=dict(workload=workload_text(cfg, head_tau, n_total),
                        tau=head_tau, hit_rate=round(head["hit_rate"], 4), l2="inputs_exceed_l2" if cfg.N * cfg.d * 2 > 126e6 else "corpus_fits_l2",
                        parallelism=f"row shards x{world} ({cfg.N} rows each), cache replicated" if sharded else f"replica x{world}", rho=args.rho, metric=args.metric,
                        cache="flat" if args.lsh_bits < 0 else f"lsh L={args.lsh_bits} b={args.lsh_bucket}", seed=args.seed, gen_seconds=round(t_gen, 1)),
            clocks=head["clocks"],
            e2e=dict(value=round(e2e, 1), unit=UNIT, h2d_bytes_per_step=head["h2d"], d2h_bytes_per_step=head["d2h"]),
            gpu_launches=int(head["launches"]),
            roofline=roof, tau_sweep=sweep_rows(cfg, results, K, peaks), cpu_baseline=cpu,
            stats=head["stats"],
        )
        line.update(extra)
        if "ms_replayed" in head:
            mr = head["ms_replayed"]
            line["replayed"] = dict(value=round(K * cfg.batch / (mr * 1e-3), 1), unit=UNIT, ms_per_step=round(mr / K, 4),
                                    us_per_query=round(mr * 1e3 / (K * cfg.batch), 3),
                                    how="prox_record_batch once, then per step a device-to-device copy of the queries "
                                        "into the recording's buffer and prox_replay_batch; same batches, same counters")

    del corpus, queries, results
    gc.collect()
    torch.cuda.empty_cache()
    if world > 1 and plain:
        # also ONE corpus dealt to the ranks by rows (the replicas' corpora have been released)
        try:
            rec = run_shard_rows(prox, base_cfg, args, dev, local, rank, world, dist, barrier, peaks, K, Wm, head_tau)
        except Exception as e:                               # the headline must survive a failure of the extra record
            rec = dict(error=f"{type(e).__name__}: {e}"[:300])
        if rank == 0:
            line["shard_rows"] = rec
    elif extras_on and rank == 0:
        wl = {}
        for name, steps in (("tiny", 1000), ("1m", 200), ("lowhit", 24)):
            if name == cfg.name:
                continue
            try:
                wl[name] = run_extra_stream_workload(prox, name, args, dev, local, peaks, steps)
            except Exception as e:
                wl[name] = dict(error=f"{type(e).__name__}: {e}"[:300])
        try:
            wl["probe"] = probe_points(prox, args, dev, local, peaks, steps=30, warmup=3)
        except Exception as e:
            wl["probe"] = dict(error=f"{type(e).__name__}: {e}"[:300])
        line["workloads"] = wl

    if rank == 0:
        print(json.dumps(line), flush=True)
    if dist:
        dist.destroy_process_group()


def run_shard_rows(prox, cfg, args, dev, local, rank, world, dist, barrier, peaks, K, Wm, tau):
    """ONE corpus dealt to the ranks by rows (strong scaling): cache and queries replicated, every rank scans
    its rows, one all-gather of the misses' lists per batch, identical merge everywhere."""
    n_total = cfg.N
    first, count = prox.shard_rows(n_total, world, rank)
    topic_rows = W.pick_topics(n_total, cfg.n_topics, args.seed, dev)
    corpus, topic_data = W.make_corpus_shard(n_total, cfg.d, cfg.n_components, args.seed, dev, first, count, topic_rows)
    nq = min(cfg.n_queries, (K + Wm) * cfg.batch)
    queries = W.make_query_stream_from_topics(topic_data, max(nq, cfg.batch), cfg.zipf_s, cfg.sigma, args.seed)
    del topic_data
    scfg = cfg.scaled(N=count)
    results, _ = run_streams(prox, scfg, queries, [tau], K, Wm, dev, local, barrier,
                             lambda t: prox.ProxShard(corpus, first, n_total, cfg.k, cfg.capacity, t, cfg.policy),
                             peaks, e2e=False, stages=False)
    r = results[tau]
    ms, _ = aggregate_over_ranks(r["ms"], K * cfg.batch, dist, dev)
    rf = scan_roofline(scfg, r, peaks)
    return dict(scaling="strong", workload=workload_text(cfg, tau, n_total), rows_per_rank=count, value=round(K * cfg.batch / (ms * 1e-3), 1),
                unit=UNIT, ms_per_step=round(ms / K, 4), hit_rate=round(r["hit_rate"], 4),
                exchange_bytes_per_batch_per_rank=16 * cfg.batch * cfg.k, exchange="one all-gather per batch (NCCL)",
                scan_ms_per_launch=rf["ms_per_launch"], scan_frac=rf["frac"], scan_bound=rf["bound"], clocks=r["clocks"])


def run_reference(args):
    """The CPU oracle as the reference arm: rank 0 only; each step is a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    oracle.build()
    name = args.workload if args.workload not in ("auto", "probe") else "large"
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
    sample = (f"extrapolated from {2 * K} queries: per step the exact top-k of 2 queries over {rows} rows and their probe "
              f"against {cap} keys, scaled to N={cfg.N} rows and capacity={cfg.capacity}; every query counted as a miss")
    line = dict(impl="reference", metric=METRIC, value=round(value, 4), unit=UNIT, n_gpus=args.gpus, steps=K,
                warmup=args.warmup, ms_per_step=round(sec_per_query * cfg.batch * 1e3, 1), higher_is_better=True,
                scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=dict(workload=workload_text(cfg, tau), tau=tau),
                cpu_baseline=dict(value=round(value, 4), unit=UNIT, cores=cores, kind="oracle", sample=sample),
                e2e=dict(value=round(value, 4), unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                gpu_launches=0)
    print(json.dumps(line), flush=True)


def probe_points(prox, args, dev, local, peaks, steps, warmup, max_keys=0):
    """Probe-only workload: a cache pre-filled with C keys, batches of 1024 queries (half near
    random keys, half fresh mixture draws), tau = 0.5; times probe + resolve + key insertion
    (prox_probe_batch) per cache size and policy, and the LSH cache at the paper's setting."""
    B, d, tau = 1024, 768, 0.5
    K = steps
    sizes = [c for c in W.PROBE_SIZES if c <= (max_keys or W.PROBE_SIZES[-1])]
    fp64_peak = 148 * 64 * 1.965e9                      # DADD/DFMA issue slots per second (64 per SM and clock)
    out = []
    for C in sizes:
        keys, centres = W.make_probe_keys(C, d, 4096, args.seed, dev)
        batches = [W.make_probe_batch(keys, centres, B, 0.02, args.seed, b) for b in range(K + warmup)]
        for policy in ("lru", "fifo"):
            p = prox.Prox(keys[:64].contiguous(), 1, C, tau, policy)
            p.cache_load(keys)
            sampler = ClockSampler(local).start()
            for q in batches[K:]:
                p.probe_batch(q)
            torch.cuda.synchronize()
            p.cache_load(keys)
            p.profile(None)
            p.profile_read()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            hits = []
            l0 = p.kernel_launches()
            sampler.begin()
            e0.record()
            for q in batches[:K]:
                hits.append(p.probe_batch(q)[0])
            e1.record()
            torch.cuda.synchronize()
            sampler.end()
            clocks = sampler.stop()
            prof = p.profile_read()
            assert p.status() == prox.OK, prox.last_error()
            ms = e0.elapsed_time(e1) / K
            hit_rate = float(torch.stack(hits).float().mean().item())
            key_bytes = C * d * 4
            t = ms * 1e-3
            flops = 2.0 * B * C * d
            # the whole batch (at-risk selection, probe, resolve, insertion) against min(HBM, tensor) of the key scan
            t_hbm, t_tc = key_bytes / (peaks["hbm_gbs"] * 1e9), flops / (peaks["bf16_tflops"] * 1e12)
            coarse = (B * C >= 2 * (1 << 20)) and C >= 4096      # the library probes large caches on the tensor cores first
            if coarse:
                roof = dict(bound="tensor", achieved=round(flops / t / 1e12, 2), peak=peaks["bf16_tflops"], unit="TFLOP/s",
                            frac=round(max(t_tc, t_hbm) / t, 4), traffic=None, kernel="scan_tc_kernel over the bf16 keys + fp64 recheck",
                            peak_kind="burst bf16 GEMM", frac_of_sustained_peak=round(flops / t / 1e12 / peaks["bf16_tflops_sustained"], 4))
            else:                                       # fp64 difference form: one subtraction, one fused multiply-add per element
                roof = dict(bound="alu", achieved=round(flops / t / 1e12, 2), peak=round(fp64_peak / 1e12, 2), unit="T fp64 instr/s",
                            frac=round(flops / t / fp64_peak, 4), traffic=None, kernel="probe_kernel")
            out.append(dict(C=C, policy=policy, us_per_batch=round(ms * 1e3, 1), keys_GBps=round(key_bytes / ms / 1e6, 1),
                            hit_rate=round(hit_rate, 4), queries_per_s=round(B / ms * 1e3, 1),
                            probe_us=round(prof["probe"][0] / K * 1e3, 1), resolve_us=round(prof["resolve"][0] / K * 1e3, 1),
                            candidates_us=round(prof["candidates"][0] / K * 1e3, 1),
                            risk_select_us=round(prof["risk_select"][0] / K * 1e3, 1),
                            gpu_launches_per_batch=round((p.kernel_launches() - l0) / K, 1),
                            probe_uncertified=p.stats()["probe_uncertified"],
                            l2="keys_exceed_l2" if key_bytes > 126e6 else "keys_fit_l2", clocks=clocks, roofline=roof))
            p.close()
        del keys, batches
        gc.collect()
        torch.cuda.empty_cache()
    # PROXIMITY-LSH at the paper's setting (L = 10, b = 20, capacity 20 480): filled by a pass of keys, then timed
    lsh = None
    if not max_keys or max_keys >= 20480:
        Lb, bb = 10, 20
        keys, centres = W.make_probe_keys(1 << 15, d, 4096, args.seed, dev)
        planes = torch.randn(Lb, d, device=dev, generator=torch.Generator(device=dev).manual_seed(args.seed + 77))
        p = prox.Prox(keys[:64].contiguous(), 1, (1 << Lb) * bb, tau, "lru", lsh_planes=planes, lsh_bucket=bb)
        for a in range(0, keys.shape[0], B):
            p.probe_batch(keys[a:a + B])
        batches = [W.make_probe_batch(keys, centres, B, 0.02, args.seed, b_) for b_ in range(K + warmup)]
        sampler = ClockSampler(local).start()
        for q in batches[K:]:
            p.probe_batch(q)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        hits = []
        sampler.begin()
        e0.record()
        for q in batches[:K]:
            hits.append(p.probe_batch(q)[0])
        e1.record()
        torch.cuda.synchronize()
        sampler.end()
        clocks = sampler.stop()
        assert p.status() == prox.OK, prox.last_error()
        ms = e0.elapsed_time(e1) / K
        st = p.stats()
        alg_bytes = B * (Lb + bb) * d * 4                  # every query reads the hyperplanes and its bucket's keys
        lsh = dict(L=Lb, b=bb, capacity=(1 << Lb) * bb, held=st["count"], us_per_batch=round(ms * 1e3, 1),
                   queries_per_s=round(B / ms * 1e3, 1), hit_rate=round(float(torch.stack(hits).float().mean().item()), 4),
                   clocks=clocks,
                   roofline=dict(bound="hbm", achieved=round(alg_bytes / ms / 1e6, 1), peak=peaks["hbm_gbs"], unit="GB/s",
                                 frac=round(alg_bytes / ms / 1e6 / peaks["hbm_gbs"], 4), traffic=None,
                                 kernel="lsh_resolve_kernel (gather of one bucket per query, replay in order)"))
        p.close()
    return dict(workload=f"probe-only: B={B} d={d} tau={tau} keys from a 4096-component mixture, full cache, LRU and FIFO",
                steps=K, warmup=warmup, points=out, lsh=lsh)


def run_probe(args):
    """`--workload probe`: the probe-only points alone, as one JSON line whose headline is the largest cache."""
    from paper_2503_05530_b200 import prox
    import __graft_entry__ as g
    g.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    peaks = load_peaks()
    K = args.steps if args.steps > 0 else 50
    res = probe_points(prox, args, dev, 0, peaks, K, args.warmup, max_keys=args.rows)
    big = res["points"][-1]
    print(json.dumps(dict(metric="probe_keys_scanned", value=big["keys_GBps"], unit="GB/s", n_gpus=1, steps=K,
                          warmup=args.warmup, ms_per_step=round(big["us_per_batch"] / 1e3, 4), higher_is_better=True,
                          scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                          config=dict(workload=res["workload"] + f"; headline C={big['C']} policy={big['policy']}", l2=big["l2"]),
                          roofline=big["roofline"], clocks=big["clocks"],
                          points=res["points"], lsh=res["lsh"])), flush=True)


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
    ap.add_argument("--default-steps", type=int, default=100, help="cap of the timed batches when --steps is 0 (a whole query stream if it is shorter)")
    ap.add_argument("--sustained-steps", type=int, default=300, help="batches of the long run of the headline tolerance")
    ap.add_argument("--sustained", action="store_true", help="add the long run also when a workload was named")
    ap.add_argument("--no-extras", action="store_true", help="headline workload only (no `workloads`, `sustained` or `shard_rows` records)")
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
