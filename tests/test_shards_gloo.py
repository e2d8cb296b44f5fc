"""Row shards on two CPU ranks over gloo: the split of the rows, the exchange step of the binding
(one all-gather of fixed-size records) and the property the merge rests on: the k nearest rows of
the whole corpus are the k smallest (distance, id) pairs among the shards' own k nearest.  The
records are filled by the oracle here; the CUDA kernels that fill and merge them are checked
against the oracle in the GPU tests."""
import os
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def make_record(ids, dists, B, k, n_miss):
    """The documented record: B*k fp64 distances, then B*k int64 ids; (+inf, -1) beyond the misses."""
    dd = np.full(B * k, np.inf, np.float64)
    ii = np.full(B * k, -1, np.int64)
    dd[:n_miss * k] = dists.ravel()
    ii[:n_miss * k] = ids.ravel()
    return np.concatenate([dd.view(np.uint8), ii.view(np.uint8)])


def merge_records(gathered, G, B, k, n_miss):
    rec = gathered.reshape(G, 16 * B * k)
    dd = np.stack([rec[g, :8 * B * k].view(np.float64).reshape(B, k) for g in range(G)], 1)   # B x G x k
    ii = np.stack([rec[g, 8 * B * k:].view(np.int64).reshape(B, k) for g in range(G)], 1)
    out_i, out_d = np.empty((n_miss, k), np.int64), np.empty((n_miss, k), np.float64)
    for m in range(n_miss):
        d, i = dd[m].ravel(), ii[m].ravel()
        order = np.lexsort((i, d))[:k]
        out_i[m], out_d[m] = i[order], d[order]
    return out_i, out_d


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2503_05530_b200 import prox, workloads as W
    N, d, k, B, n_miss = 1001, 32, 7, 12, 9
    X = W.make_corpus(N, d, 8, 3, "cpu")
    X[500:520] = X[100:120]                                   # equal rows in different shards: ties by id
    Q, _, _ = W.make_query_stream(X, n_miss, 5, 1.0, 0.05, 3)
    first, cnt = prox.shard_rows(N, world, rank)
    ids, dists = oracle.exact_topk(X[first:first + cnt].numpy(), Q.numpy(), k)
    record = torch.from_numpy(make_record(ids + first, dists, B, k, n_miss))
    gathered = prox.all_gather_records(record)
    assert gathered.numel() == world * record.numel()
    got_i, got_d = merge_records(gathered.numpy(), world, B, k, n_miss)
    ref_i, ref_d = oracle.exact_topk(X.numpy(), Q.numpy(), k)
    same = bool(np.array_equal(got_i, ref_i) and np.array_equal(got_d, ref_d))
    digest = torch.tensor([float(got_i.sum()), float(got_d.sum())], dtype=torch.float64)
    both = [torch.zeros(2, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(both, digest)
    if rank == 0:
        out.put((same, [b.tolist() for b in both], (first, cnt)))
    dist.barrier()
    dist.destroy_process_group()


def test_two_shards_exchange_and_merge_to_the_whole_corpus_result():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    same, digests, rows0 = out.get(timeout=180)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert same, "merged shard results differ from the exact top-k of the whole corpus"
    assert digests[0] == digests[1], "both ranks must arrive at the same lists"
    assert rows0 == (0, 501)


def _rank_stream(rank, world, port, out):
    """A stream of several batches: the cache is replicated (its decisions depend on the queries
    alone, so every rank replays the same trace without talking to anyone), each batch's misses
    are answered from the shards' own nearest rows through one exchange, and the merged lists
    are what later hits return."""
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import oracle
    from paper_2503_05530_b200 import prox, workloads as W
    N, d, k, B, n, cap, tau = 1503, 32, 5, 16, 112, 6, 0.3
    X = W.make_corpus(N, d, 8, 4, "cpu")
    X[700:710] = X[20:30]                                     # equal rows in different shards
    Q, _, _ = W.make_query_stream(X, n, 40, 1.0, 0.05, 4)
    Xn, Qn = X.numpy(), Q.numpy()
    first, cnt = prox.shard_rows(N, world, rank)
    trace = oracle.Oracle(None, d, k, cap, float(np.float32(tau)), oracle.LRU)
    lists, out_ids, out_hit = {}, np.empty((n, k), np.int64), np.empty(n, np.uint8)
    for a in range(0, n, B):
        r = trace.query(Qn[a:a + B])
        miss = np.nonzero(r["hit"] == 0)[0]
        if len(miss):
            ids, dists = oracle.exact_topk(Xn[first:first + cnt], Qn[a:a + B][miss], k)
        else:
            ids, dists = np.empty((0, k), np.int64), np.empty((0, k), np.float64)
        record = torch.from_numpy(make_record(ids + first, dists, B, k, len(miss)))
        gathered = prox.all_gather_records(record)            # the one exchange of the batch
        got_i, _ = merge_records(gathered.numpy(), world, B, k, len(miss))
        for j, m in enumerate(miss):
            lists[a + int(m)] = got_i[j]
        for i in range(B):
            out_ids[a + i] = lists[int(r["origin"][i])]        # a hit returns the list of the miss that made its key
            out_hit[a + i] = r["hit"][i]
    whole = oracle.Oracle(Xn, d, k, cap, float(np.float32(tau)), oracle.LRU).query(Qn)
    same = bool(np.array_equal(out_ids, whole["ids"]) and np.array_equal(out_hit, whole["hit"]))
    digest = torch.tensor([float(out_ids.sum()), float(out_hit.sum())], dtype=torch.float64)
    both = [torch.zeros(2, dtype=torch.float64) for _ in range(world)]
    dist.all_gather(both, digest)
    if rank == 0:
        out.put((same, [b.tolist() for b in both], float(whole["hit"].mean()), int((whole["evicted"] >= 0).sum())))
    dist.barrier()
    dist.destroy_process_group()


def test_two_shards_carry_a_stream_of_batches():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 33500 + os.getpid() % 2000
    procs = [ctx.Process(target=_rank_stream, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    same, digests, hit_rate, evictions = out.get(timeout=180)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert same, "the sharded stream differs from the oracle on the whole corpus"
    assert digests[0] == digests[1], "both ranks must end with the same lists and flags"
    assert 0.2 < hit_rate < 0.95 and evictions > 0


def test_shard_rows_cover_the_corpus_once():
    from paper_2503_05530_b200 import prox
    for n, g in [(10, 3), (7, 7), (24_000_000, 8), (5, 1), (100, 32)]:
        spans = [prox.shard_rows(n, g, r) for r in range(g)]
        assert spans[0][0] == 0 and sum(c for _, c in spans) == n
        for (a, ca), (b, _) in zip(spans, spans[1:]):
            assert a + ca == b
        assert max(c for _, c in spans) - min(c for _, c in spans) <= 1


def test_all_gather_without_a_process_group_is_the_record_itself():
    from paper_2503_05530_b200 import prox
    r = torch.arange(32, dtype=torch.uint8)
    assert prox.all_gather_records(r) is r


def test_shard_generator_draws_the_rows_of_the_whole_corpus():
    from paper_2503_05530_b200 import prox, workloads as W
    N, d = 1003, 16
    X = W.make_corpus(N, d, 8, 3, "cpu", chunk_rows=100)
    Q, _, rows = W.make_query_stream(X, 60, 25, 1.0, 0.05, 3)
    for g in range(3):
        first, cnt = prox.shard_rows(N, 3, g)
        shard, kept = W.make_corpus_shard(N, d, 8, 3, "cpu", first, cnt, rows, chunk_rows=100)
        assert torch.equal(shard, X[first:first + cnt]) and torch.equal(kept, X[rows])
        assert torch.equal(W.make_query_stream_from_topics(kept, 60, 1.0, 0.05, 3), Q)
