"""Two CPU ranks over gloo: the whole-job aggregation that `bench.py --gpus N` reports
(slowest rank's time, queries of all ranks) and the per-rank stream seeds."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    from paper_2503_05530_b200 import workloads as W
    ms, total = bench.aggregate_over_ranks(10.0 + 5.0 * rank, 100 * (rank + 1), dist, "cpu")
    # every rank builds the same index and draws its own query stream
    X = W.make_corpus(300, 32, 4, 0, "cpu")
    Q, _, _ = W.make_query_stream(X, 16, 10, 1.1, 0.02, bench.stream_seed(0, rank))
    sums = [torch.zeros(2, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(sums, torch.tensor([float(X.double().sum()), float(Q.double().sum())], dtype=torch.float64))
    if rank == 0:
        out.put((ms, total, [s.tolist() for s in sums]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_aggregate_max_time_and_sum_of_queries():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    ms, total, sums = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert ms == 15.0 and total == 300
    assert sums[0][0] == sums[1][0], "the corpus must be the same on every rank"
    assert sums[0][1] != sums[1][1], "every rank must serve its own query stream"


def test_single_process_aggregate_is_identity():
    import bench
    assert bench.aggregate_over_ranks(3.5, 7) == (3.5, 7)
