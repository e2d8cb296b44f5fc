"""ctypes binding of the CUDA library (``libprox.so``): argument marshalling only.

Every step of a lookup runs in the library's kernels; this module converts
tensors to pointers and sizes.  It raises if the library has not been built:
there is no CPU path.  PyTorch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libprox.so")

LRU, FIFO = 0, 1
OK, ERR_INVALID_ARG, ERR_OOM, ERR_CUDA, ERR_UNSUPPORTED, ERR_TIMEOUT, ERR_INTERNAL = range(7)
MAX_K, MAX_BATCH = 64, 1024
SCAN_AUTO, SCAN_CUDA_CORE, SCAN_TC_SINGLE = 0, 1, 2
STAGES = ("risk_select", "probe", "candidates", "resolve", "gather", "prep_miss", "scan", "merge",
          "rerank", "exact_pass", "scatter")
_POLICY = {"lru": LRU, "fifo": FIFO, LRU: LRU, FIFO: FIFO}
METRIC_L2SQ, METRIC_COSINE, METRIC_IP = 0, 1, 2
_METRIC = {"l2": METRIC_L2SQ, "cosine": METRIC_COSINE, "ip": METRIC_IP, METRIC_L2SQ: METRIC_L2SQ,
           METRIC_COSINE: METRIC_COSINE, METRIC_IP: METRIC_IP}


class ProxError(RuntimeError):
    pass


class Stats(C.Structure):
    _fields_ = [(n, C.c_int64) for n in ("queries", "hits", "misses", "intra_batch_hits", "evictions",
                                          "scan_batches", "uncertified", "fallback_rows", "unresolved",
                                          "count", "probe_uncertified", "parallel_replays")]

    def as_dict(self) -> dict:
        return {n: int(getattr(self, n)) for n, _ in self._fields_}


_lib = None


def load_library():
    """dlopen the CUDA library; fails loudly if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ProxError(f"{LIB_PATH} is not built: run `python -c 'import __graft_entry__ as g; g.build()'` "
                        "(there is no CPU fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    L.prox_create.restype = vp
    L.prox_create.argtypes = [vp, i64, i32, i32, i64, f32, i32]
    L.prox_create_rho.restype = vp
    L.prox_create_rho.argtypes = [vp, i64, i32, i32, i64, f32, i32, i32]
    L.prox_create_metric.restype = vp
    L.prox_create_metric.argtypes = [vp, i64, i32, i32, i64, f32, i32, i32, i32]
    L.prox_create_lsh.restype = vp
    L.prox_create_lsh.argtypes = [vp, i64, i32, i32, i32, i32, vp, f32, i32, i32]
    L.prox_query_batch.restype = i32
    L.prox_query_batch.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    L.prox_create_shard.restype = vp
    L.prox_create_shard.argtypes = [vp, i64, i32, i32, i64, f32, i32, i32, i64, i64]
    L.prox_shard_exchange_bytes.restype = i64
    L.prox_shard_exchange_bytes.argtypes = [vp, i32]
    L.prox_shard_scan.restype = i32
    L.prox_shard_scan.argtypes = [vp, vp, i32, vp, vp, vp, vp, vp]
    L.prox_shard_merge.restype = i32
    L.prox_shard_merge.argtypes = [vp, vp, i32, vp, i32, vp, vp, vp]
    L.prox_query_batch_host.restype = i32
    L.prox_query_batch_host.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    L.prox_reset_cache.restype = i32
    L.prox_reset_cache.argtypes = [vp, vp]
    L.prox_destroy.restype = None
    L.prox_destroy.argtypes = [vp]
    L.prox_last_error.restype = C.c_char_p
    L.prox_cache_load.restype = i32
    L.prox_cache_load.argtypes = [vp, vp, i64, vp]
    L.prox_probe_batch.restype = i32
    L.prox_probe_batch.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    L.prox_get_stats.restype = i32
    L.prox_get_stats.argtypes = [vp, C.POINTER(Stats), vp]
    L.prox_status.restype = i32
    L.prox_status.argtypes = [vp, vp]
    L.prox_set_scan_mode.restype = i32
    L.prox_set_scan_mode.argtypes = [vp, i32]
    L.prox_kernel_launches.restype = i64
    L.prox_kernel_launches.argtypes = [vp]
    L.prox_profile.restype = i32
    L.prox_profile.argtypes = [vp, C.c_uint32]
    L.prox_profile_read.restype = i32
    L.prox_profile_read.argtypes = [vp, C.POINTER(C.c_double), C.POINTER(i64), vp]
    L.prox_record_batch.restype = vp
    L.prox_record_batch.argtypes = [vp, vp, i32, vp, vp, vp, vp]
    L.prox_replay_batch.restype = i32
    L.prox_replay_batch.argtypes = [vp, vp]
    L.prox_recorded_batch_destroy.restype = None
    L.prox_recorded_batch_destroy.argtypes = [vp]
    L.prox_nearest_key_static.restype = i32
    L.prox_nearest_key_static.argtypes = [vp, i64, i32, vp, i32, vp, vp, vp]
    _lib = L
    return L


def last_error() -> str:
    return load_library().prox_last_error().decode()


def _check(rc: int):
    if rc != OK:
        raise ProxError(f"prox error {rc}: {last_error()}")


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev_f32(t: torch.Tensor, what: str) -> torch.Tensor:
    if not (t.is_cuda and t.dtype == torch.float32 and t.is_contiguous() and t.dim() == 2):
        raise ProxError(f"{what} must be a contiguous 2-d float32 CUDA tensor")
    return t


def nearest_key_static(keys: torch.Tensor, queries: torch.Tensor, out_slot: torch.Tensor, out_dist: torch.Tensor,
                       stream=None):
    """prox_nearest_key_static: nearest key per query, for callers that may not allocate device memory.
    Every tensor is the caller's (CUDA, contiguous; keys/queries float32, out_slot int32, out_dist float32);
    the binding allocates nothing either."""
    _check(load_library().prox_nearest_key_static(keys.data_ptr(), keys.shape[0], keys.shape[1], queries.data_ptr(),
                                                  queries.shape[0], out_slot.data_ptr(), out_dist.data_ptr(),
                                                  _stream_ptr(stream)))


class RecordedBatch:
    """A recorded prox_query_batch call (prox_record_batch); keeps its buffers alive."""

    def __init__(self, owner, ptr, buffers):
        self._owner, self._r, self.buffers = owner, ptr, buffers

    def replay(self, stream=None):
        _check(self._owner._lib.prox_replay_batch(self._r, _stream_ptr(stream)))

    def close(self):
        if self._r:
            self._owner._lib.prox_recorded_batch_destroy(self._r)
            self._r = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Prox:
    """prox_create / prox_query_batch / prox_reset_cache / prox_destroy with tensors."""

    def __init__(self, corpus: torch.Tensor, k: int, capacity: int, tau: float, policy="lru", rho: int = 1,
                 lsh_planes: torch.Tensor | None = None, lsh_bucket: int = 0, metric="l2"):
        self._lib = load_library()
        self._corpus = _dev_f32(corpus, "corpus")      # borrowed by the library: keep it alive
        self.N, self.d = corpus.shape
        self.k, self.capacity, self.tau = int(k), int(capacity), float(tau)
        self.policy = _POLICY[policy]
        self.rho = int(rho)                            # re-ranking factor (prox_create_rho); 1 = prox_create
        with torch.cuda.device(corpus.device):
            self.metric = _METRIC[metric]
            if lsh_planes is None:
                self._h = self._lib.prox_create_metric(corpus.data_ptr(), self.N, self.d, self.k, self.capacity,
                                                       self.tau, self.policy, self.rho, self.metric)
            elif self.metric != METRIC_L2SQ:
                raise ProxError("PROXIMITY-LSH handles take the Euclidean distance only")
            else:
                # PROXIMITY-LSH (prox_create_lsh): 2^L buckets of lsh_bucket entries; capacity = 2^L * lsh_bucket
                P = _dev_f32(lsh_planes.reshape(-1, self.d), "lsh_planes")
                L_ = P.shape[0]
                if self.capacity != (1 << L_) * lsh_bucket:
                    raise ProxError("capacity must equal 2^L * lsh_bucket")
                self._h = self._lib.prox_create_lsh(corpus.data_ptr(), self.N, self.d, self.k, L_, int(lsh_bucket),
                                                    P.data_ptr() if L_ else None, self.tau, self.policy, self.rho)
        if not self._h:
            raise ProxError(f"prox_create failed: {last_error()}")
        self.device = corpus.device

    def close(self):
        if getattr(self, "_h", None):
            self._lib.prox_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *a):
        self.close()

    def query_batch(self, queries: torch.Tensor, out_ids=None, out_dists=None, out_hit=None, stream=None):
        q = _dev_f32(queries, "queries")
        B = q.shape[0]
        if q.shape[1] != self.d:
            raise ProxError("queries have the wrong dimension")
        if out_ids is None:
            out_ids = torch.empty(B, self.k, dtype=torch.int64, device=self.device)
        if out_dists is None:
            out_dists = torch.empty(B, self.k, dtype=torch.float32, device=self.device)
        if out_hit is None:
            out_hit = torch.empty(B, dtype=torch.uint8, device=self.device)
        _check(self._lib.prox_query_batch(self._h, q.data_ptr(), B, out_ids.data_ptr(), out_dists.data_ptr(),
                                          out_hit.data_ptr(), _stream_ptr(stream)))
        return out_ids, out_dists, out_hit

    def record_batch(self, queries: torch.Tensor, out_ids: torch.Tensor, out_dists: torch.Tensor,
                     out_hit: torch.Tensor, stream=None) -> "RecordedBatch":
        """prox_record_batch: the batch call on these buffers as a replayable recording (nothing runs
        yet).  `stream` (default: the current one) must not be the legacy default stream."""
        q = _dev_f32(queries, "queries")
        if q.shape[1] != self.d:
            raise ProxError("queries have the wrong dimension")
        B = q.shape[0]
        for t, dt in ((out_ids, torch.int64), (out_dists, torch.float32), (out_hit, torch.uint8)):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == dt and t.shape[0] == B):
                raise ProxError("record_batch takes contiguous CUDA outputs of the batch's shape")
        r = self._lib.prox_record_batch(self._h, q.data_ptr(), B, out_ids.data_ptr(), out_dists.data_ptr(),
                                        out_hit.data_ptr(), _stream_ptr(stream))
        if not r:
            raise ProxError(f"prox_record_batch failed: {last_error()}")
        return RecordedBatch(self, r, (q, out_ids, out_dists, out_hit))

    def query_batch_host(self, queries: torch.Tensor, out_ids: torch.Tensor, out_dists: torch.Tensor,
                         out_hit: torch.Tensor, stream=None):
        """Host tensors in and out (pinned for speed); synchronises the stream."""
        B = queries.shape[0]
        for t in (queries, out_ids, out_dists, out_hit):
            if t.is_cuda or not t.is_contiguous():
                raise ProxError("query_batch_host takes contiguous host tensors")
        _check(self._lib.prox_query_batch_host(self._h, queries.data_ptr(), B, out_ids.data_ptr(),
                                               out_dists.data_ptr(), out_hit.data_ptr(), _stream_ptr(stream)))
        return out_ids, out_dists, out_hit

    def probe_batch(self, queries: torch.Tensor, stream=None):
        q = _dev_f32(queries, "queries")
        B = q.shape[0]
        hit = torch.empty(B, dtype=torch.uint8, device=self.device)
        slot = torch.empty(B, dtype=torch.int32, device=self.device)
        dist = torch.empty(B, dtype=torch.float32, device=self.device)
        _check(self._lib.prox_probe_batch(self._h, q.data_ptr(), B, hit.data_ptr(), slot.data_ptr(),
                                          dist.data_ptr(), _stream_ptr(stream)))
        return hit, slot, dist

    def cache_load(self, keys: torch.Tensor, stream=None):
        kk = _dev_f32(keys, "keys")
        if kk.shape[1] != self.d:
            raise ProxError("keys have the wrong dimension")
        _check(self._lib.prox_cache_load(self._h, kk.data_ptr(), kk.shape[0], _stream_ptr(stream)))

    def reset_cache(self, stream=None):
        _check(self._lib.prox_reset_cache(self._h, _stream_ptr(stream)))

    def stats(self, stream=None) -> dict:
        st = Stats()
        _check(self._lib.prox_get_stats(self._h, C.byref(st), _stream_ptr(stream)))
        return st.as_dict()

    def status(self, stream=None) -> int:
        return int(self._lib.prox_status(self._h, _stream_ptr(stream)))

    def set_scan_mode(self, mode: int):
        _check(self._lib.prox_set_scan_mode(self._h, mode))

    def kernel_launches(self) -> int:
        return int(self._lib.prox_kernel_launches(self._h))

    def profile(self, stages=None):
        """Record CUDA events around the named stages (None = all, () = off)."""
        if stages is None:
            mask = (1 << len(STAGES)) - 1
        else:
            mask = 0
            for name in stages:
                mask |= 1 << STAGES.index(name)
        _check(self._lib.prox_profile(self._h, mask))

    def profile_read(self, stream=None) -> dict:
        """{stage: (milliseconds, launches)} since the last read; synchronises the stream."""
        ms = (C.c_double * len(STAGES))()
        n = (C.c_int64 * len(STAGES))()
        _check(self._lib.prox_profile_read(self._h, ms, n, _stream_ptr(stream)))
        return {name: (float(ms[i]), int(n[i])) for i, name in enumerate(STAGES)}


def shard_rows(n_total: int, n_shards: int, shard: int) -> tuple[int, int]:
    """Rows [first, first + count) of shard `shard` when n_total rows are dealt to n_shards GPUs in
    contiguous runs whose lengths differ by at most one (the longer runs first)."""
    if not (0 <= shard < n_shards):
        raise ProxError("shard index out of range")
    base, extra = divmod(int(n_total), int(n_shards))
    first = shard * base + min(shard, extra)
    return first, base + (1 if shard < extra else 0)


def all_gather_records(record: torch.Tensor, group=None) -> torch.Tensor:
    """The one exchange step of a row-sharded lookup: every rank contributes its exchange record
    (a 1-d uint8 tensor of equal length on every rank) and receives all of them back to back, in
    rank order.  Without an initialised process group (or with a group of one) the record is its
    own gathering."""
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size(group) == 1:
        return record
    G = dist.get_world_size(group)
    out = torch.empty(G * record.numel(), dtype=record.dtype, device=record.device)
    dist.all_gather_into_tensor(out, record, group=group)
    return out


class ProxShard(Prox):
    """One row shard of a corpus split over several GPUs (prox_create_shard / prox_shard_scan /
    prox_shard_merge).  Every rank holds the rows shard_rows(n_total, G, rank) and calls
    query_batch with the same queries; the cache is replicated and needs no exchange."""

    def __init__(self, corpus_shard: torch.Tensor, row_offset: int, n_total: int, k: int, capacity: int, tau: float,
                 policy="lru", metric="l2", group=None):
        self._lib = load_library()
        self._corpus = _dev_f32(corpus_shard, "corpus_shard")
        self.N, self.d = corpus_shard.shape
        self.k, self.capacity, self.tau = int(k), int(capacity), float(tau)
        self.policy, self.rho, self.metric = _POLICY[policy], 1, _METRIC[metric]
        self.row_offset, self.n_total, self.group = int(row_offset), int(n_total), group
        with torch.cuda.device(corpus_shard.device):
            self._h = self._lib.prox_create_shard(corpus_shard.data_ptr(), self.N, self.d, self.k, self.capacity,
                                                  self.tau, self.policy, self.metric, self.row_offset, self.n_total)
        if not self._h:
            raise ProxError(f"prox_create_shard failed: {last_error()}")
        self.device = corpus_shard.device

    def exchange_bytes(self, B: int) -> int:
        return int(self._lib.prox_shard_exchange_bytes(self._h, B))

    def shard_scan(self, queries: torch.Tensor, out_ids, out_dists, out_hit, record: torch.Tensor, stream=None):
        q = _dev_f32(queries, "queries")
        if q.shape[1] != self.d or record.numel() * record.element_size() < self.exchange_bytes(q.shape[0]):
            raise ProxError("queries have the wrong dimension or the record is too small")
        _check(self._lib.prox_shard_scan(self._h, q.data_ptr(), q.shape[0], out_ids.data_ptr(), out_dists.data_ptr(),
                                         out_hit.data_ptr(), record.data_ptr(), _stream_ptr(stream)))

    def shard_merge(self, queries: torch.Tensor, gathered: torch.Tensor, n_shards: int, out_ids, out_dists, stream=None):
        B = queries.shape[0]
        if gathered.numel() * gathered.element_size() < n_shards * self.exchange_bytes(B):
            raise ProxError("gathered holds fewer than n_shards records")
        _check(self._lib.prox_shard_merge(self._h, queries.data_ptr(), B, gathered.data_ptr(), int(n_shards),
                                          out_ids.data_ptr(), out_dists.data_ptr(), _stream_ptr(stream)))

    def query_batch(self, queries: torch.Tensor, out_ids=None, out_dists=None, out_hit=None, stream=None):
        """Scan of this shard, all-gather of the records over the process group, merge."""
        B = queries.shape[0]
        if out_ids is None:
            out_ids = torch.empty(B, self.k, dtype=torch.int64, device=self.device)
        if out_dists is None:
            out_dists = torch.empty(B, self.k, dtype=torch.float32, device=self.device)
        if out_hit is None:
            out_hit = torch.empty(B, dtype=torch.uint8, device=self.device)
        # the exchange is ordered on the stream the two library calls use: torch orders a collective after
        # the work already queued on the CURRENT stream and makes that stream wait for its result
        with torch.cuda.stream(stream if stream is not None else torch.cuda.current_stream()):
            record = torch.empty(self.exchange_bytes(B), dtype=torch.uint8, device=self.device)
            self.shard_scan(queries, out_ids, out_dists, out_hit, record, stream)
            gathered = all_gather_records(record, self.group)
            self.shard_merge(queries, gathered, gathered.numel() // record.numel(), out_ids, out_dists, stream)
        return out_ids, out_dists, out_hit

    def query_batch_host(self, queries: torch.Tensor, out_ids: torch.Tensor, out_dists: torch.Tensor,
                         out_hit: torch.Tensor, stream=None):
        """Host tensors in and out (pinned for speed): copies on the current stream around
        query_batch, then synchronises.  Every rank passes the same queries."""
        B = queries.shape[0]
        for t in (queries, out_ids, out_dists, out_hit):
            if t.is_cuda or not t.is_contiguous():
                raise ProxError("query_batch_host takes contiguous host tensors")
        if getattr(self, "_stage", None) is None:
            MB = MAX_BATCH
            self._stage = (torch.empty(MB, self.d, dtype=torch.float32, device=self.device),
                           torch.empty(MB, self.k, dtype=torch.int64, device=self.device),
                           torch.empty(MB, self.k, dtype=torch.float32, device=self.device),
                           torch.empty(MB, dtype=torch.uint8, device=self.device))
        q, ids, dists, hit = (t[:B] for t in self._stage)
        with torch.cuda.stream(stream if stream is not None else torch.cuda.current_stream()):
            q.copy_(queries, non_blocking=True)
            self.query_batch(q, ids, dists, hit)
            out_ids.copy_(ids, non_blocking=True)
            out_dists.copy_(dists, non_blocking=True)
            out_hit.copy_(hit, non_blocking=True)
            torch.cuda.current_stream().synchronize()
        return out_ids, out_dists, out_hit
