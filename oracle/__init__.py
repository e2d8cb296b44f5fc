"""TEST INFRASTRUCTURE: ctypes front end of the fp64 CPU oracle (``prox_oracle.c``).

The oracle restates Algorithm 1 of the paper (cache lookup in PROXIMITY-FLAT),
its eviction policies (Section 3.3.2) and the exact top-k database call in plain
sequential C.  It exists so that the CUDA library can be checked against
something that was written from the paper alone; it imports nothing from the
CUDA package and the CUDA package never imports it.  Only tests, the smoke
check and the CPU-baseline leg of the benchmark may call it.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "prox_oracle.c")
_LIB = os.path.join(_HERE, "_prox_oracle.so")

LRU, FIFO = 0, 1
L2SQ, COSINE, IP = 0, 1, 2


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fused multiply-add contraction, OpenMP over rows)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = C.CDLL(build())
        fp, ip, dp, i32p = (C.POINTER(C.c_float), C.POINTER(C.c_int64), C.POINTER(C.c_double),
                            C.POINTER(C.c_int32))
        L.oracle_num_threads.restype = C.c_int
        L.oracle_set_threads.argtypes = [C.c_int]
        L.oracle_sqdist.restype = C.c_double
        L.oracle_sqdist.argtypes = [fp, fp, C.c_int32]
        L.oracle_create.restype = C.c_void_p
        L.oracle_create.argtypes = [fp, C.c_int64, C.c_int32, C.c_int32, C.c_int64, C.c_double, C.c_int32]
        L.oracle_create_rho.restype = C.c_void_p
        L.oracle_create_rho.argtypes = [fp, C.c_int64, C.c_int32, C.c_int32, C.c_int64, C.c_double, C.c_int32, C.c_int32]
        L.oracle_create_lsh.restype = C.c_void_p
        L.oracle_create_lsh.argtypes = [fp, C.c_int64, C.c_int32, C.c_int32, C.c_int32, C.c_int32, fp, C.c_double,
                                        C.c_int32, C.c_int32]
        L.oracle_lsh_hash.restype = C.c_int64
        L.oracle_lsh_hash.argtypes = [fp, C.c_int32, C.c_int32, fp]
        L.oracle_set_metric.restype = C.c_int
        L.oracle_set_metric.argtypes = [C.c_void_p, C.c_int32]
        L.oracle_cosdist.restype = C.c_double
        L.oracle_cosdist.argtypes = [fp, fp, C.c_int32]
        L.oracle_ipdist.restype = C.c_double
        L.oracle_ipdist.argtypes = [fp, fp, C.c_int32]
        L.oracle_knn_batch_metric.argtypes = [C.c_int32, fp, C.c_int64, C.c_int32, fp, C.c_int64, C.c_int32, ip, dp]
        L.oracle_destroy.argtypes = [C.c_void_p]
        L.oracle_reset.argtypes = [C.c_void_p]
        L.oracle_counters.argtypes = [C.c_void_p, ip]
        L.oracle_cache_load.restype = C.c_int
        L.oracle_cache_load.argtypes = [C.c_void_p, fp, C.c_int64]
        L.oracle_query_stream.argtypes = [C.c_void_p, fp, C.c_int64, i32p, ip, dp, ip, dp]
        L.oracle_knn_batch.argtypes = [fp, C.c_int64, C.c_int32, fp, C.c_int64, C.c_int32, ip, dp]
        L.oracle_topk_update.argtypes = [fp, C.c_int64, C.c_int32, C.c_int64, fp, C.c_int32, dp, ip, dp, i32p]
        L.oracle_slot_stamp.restype = C.c_int64
        L.oracle_slot_stamp.argtypes = [C.c_void_p, C.c_int64]
        L.oracle_slot_origin.restype = C.c_int64
        L.oracle_slot_origin.argtypes = [C.c_void_p, C.c_int64]
        _lib = L
    return _lib


def _f32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a), dtype=np.float32)


def _ptr(a: np.ndarray, ctype):
    return a.ctypes.data_as(C.POINTER(ctype))


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_threads(n: int) -> None:
    """Threads the row loops of the database call use from now on (the arithmetic does not depend on it)."""
    lib().oracle_set_threads(int(n))


def sqdist(a, b) -> float:
    """Squared Euclidean distance in fp64 over fp32 inputs (Algorithm 1, ``distance``)."""
    a, b = _f32(a).ravel(), _f32(b).ravel()
    assert a.shape == b.shape
    return float(lib().oracle_sqdist(_ptr(a, C.c_float), _ptr(b, C.c_float), a.size))


def cosdist(a, b) -> float:
    """Cosine distance 1 - cos(a, b) in fp64 over fp32 inputs (half the squared distance of the unit vectors)."""
    a, b = _f32(a).ravel(), _f32(b).ravel()
    assert a.shape == b.shape
    return float(lib().oracle_cosdist(_ptr(a, C.c_float), _ptr(b, C.c_float), a.size))


def ipdist(a, b) -> float:
    """Inner product as a distance, -(a . b), in fp64 over fp32 inputs."""
    a, b = _f32(a).ravel(), _f32(b).ravel()
    assert a.shape == b.shape
    return float(lib().oracle_ipdist(_ptr(a, C.c_float), _ptr(b, C.c_float), a.size))


def exact_topk(corpus, queries, k: int, metric: int = L2SQ):
    """The database call alone: for each query the k nearest corpus rows, (ids[n,k], dists[n,k])."""
    X, Q = _f32(corpus), _f32(queries)
    if Q.ndim == 1:
        Q = Q[None, :]
    n, d = Q.shape
    assert X.shape[1] == d and 1 <= k <= X.shape[0]
    ids = np.empty((n, k), np.int64)
    dists = np.empty((n, k), np.float64)
    lib().oracle_knn_batch_metric(metric, _ptr(X, C.c_float), X.shape[0], d, _ptr(Q, C.c_float), n, k,
                                  _ptr(ids, C.c_int64), _ptr(dists, C.c_double))
    return ids, dists


def lsh_hash(planes, q) -> int:
    """h(q) of PROXIMITY-LSH: bit l is (q . r_l >= 0) for the l-th row of ``planes``."""
    P, v = _f32(planes), _f32(q).ravel()
    assert P.ndim == 2 and P.shape[1] == v.size
    return int(lib().oracle_lsh_hash(_ptr(P, C.c_float), P.shape[0], P.shape[1], _ptr(v, C.c_float)))


class ChunkedTopK:
    """The database call for ONE query with the corpus fed in ascending row chunks."""

    def __init__(self, query, k: int):
        self.q = _f32(query).ravel()
        self.k = k
        self.ids = np.full(k, -1, np.int64)
        self.dists = np.full(k, np.inf, np.float64)
        self.have = C.c_int32(0)
        self.next_row = 0

    def feed(self, chunk) -> None:
        X = _f32(chunk)
        assert X.shape[1] == self.q.size
        lib().oracle_topk_update(_ptr(X, C.c_float), X.shape[0], X.shape[1], self.next_row,
                                 _ptr(self.q, C.c_float), self.k, None, _ptr(self.ids, C.c_int64),
                                 _ptr(self.dists, C.c_double), C.byref(self.have))
        self.next_row += X.shape[0]


class Oracle:
    """Algorithm 1 as a sequential state machine.  ``corpus=None`` gives the cache trace only
    (hits, slots, evictions depend on the query stream alone; lists are then filled with -1).
    ``rho`` is the re-ranking factor: rho * k neighbours are fetched and stored per miss, and a
    hit returns the k of them nearest to the current query (rho = 1: the stored list as it is).
    ``lsh_planes`` (L x d) with ``lsh_bucket`` = b switches to PROXIMITY-LSH: 2^L buckets of b entries."""

    def __init__(self, corpus, d: int, k: int, capacity: int, tau: float, policy: int, rho: int = 1,
                 lsh_planes=None, lsh_bucket: int = 0, metric: int = L2SQ):
        self._X = None if corpus is None else _f32(corpus)
        N = 0 if self._X is None else self._X.shape[0]
        if self._X is not None:
            assert self._X.shape[1] == d
        self.d, self.k, self.capacity, self.tau, self.policy = d, k, capacity, float(tau), policy
        self.rho = int(rho)
        xp = None if self._X is None else _ptr(self._X, C.c_float)
        if lsh_planes is None:
            self._h = lib().oracle_create_rho(xp, N, d, k, capacity, float(tau), policy, self.rho)
        else:
            # PROXIMITY-LSH: one bucket of lsh_bucket entries per hash code; capacity = 2^L * lsh_bucket
            self._P = _f32(lsh_planes).reshape(-1, d)
            L_ = self._P.shape[0]
            assert capacity == (1 << L_) * lsh_bucket, "capacity must be 2^L * bucket size"
            self._h = lib().oracle_create_lsh(xp, N, d, k, L_, lsh_bucket, _ptr(self._P, C.c_float) if L_ else None,
                                              float(tau), policy, self.rho)
        if not self._h:
            raise ValueError("oracle_create rejected the arguments")
        if lib().oracle_set_metric(self._h, metric):
            self.close()
            raise ValueError("metric unknown, or not available with these arguments (a negative tolerance goes with the "
                             "inner product only; PROXIMITY-LSH does not take the inner product)")

    def close(self):
        if self._h:
            lib().oracle_destroy(self._h)
            self._h = None

    __del__ = close

    def reset(self):
        lib().oracle_reset(self._h)

    def cache_load(self, keys):
        K = _f32(keys)
        assert K.shape[1] == self.d
        if lib().oracle_cache_load(self._h, _ptr(K, C.c_float), K.shape[0]):
            raise ValueError("more keys than capacity")

    def counters(self) -> dict:
        out = np.zeros(5, np.int64)
        lib().oracle_counters(self._h, _ptr(out, C.c_int64))
        return dict(probe_madds=int(out[0]), hits=int(out[1]), misses=int(out[2]),
                    evictions=int(out[3]), count=int(out[4]))

    def slot_stamp(self, s: int) -> int:
        return int(lib().oracle_slot_stamp(self._h, s))

    def slot_origin(self, s: int) -> int:
        return int(lib().oracle_slot_origin(self._h, s))

    def query(self, queries, force=None) -> dict:
        """Feed queries one after the other.  Returns ids[n,k] (int64), dists[n,k] (fp64),
        hit[n], slot[n], origin[n] (stream index of the query whose miss made the matched key;
        own index on a miss), evicted[n] (slot or -1), best[n], second[n] (nearest and second
        nearest key distance at the time of the lookup)."""
        Q = _f32(queries)
        if Q.ndim == 1:
            Q = Q[None, :]
        n = Q.shape[0]
        assert Q.shape[1] == self.d
        ids = np.empty((n, self.k), np.int64)
        dists = np.empty((n, self.k), np.float64)
        trace = np.empty((n, 4), np.int64)
        dtrace = np.empty((n, 2), np.float64)
        fptr = None
        if force is not None:
            force = np.ascontiguousarray(force, dtype=np.int32)
            assert force.shape == (n,)
            fptr = _ptr(force, C.c_int32)
        lib().oracle_query_stream(self._h, _ptr(Q, C.c_float), n, fptr, _ptr(ids, C.c_int64),
                                  _ptr(dists, C.c_double), _ptr(trace, C.c_int64),
                                  _ptr(dtrace, C.c_double))
        return dict(ids=ids, dists=dists, hit=trace[:, 0].astype(np.uint8), slot=trace[:, 1].copy(),
                    origin=trace[:, 2].copy(), evicted=trace[:, 3].copy(),
                    best=dtrace[:, 0].copy(), second=dtrace[:, 1].copy())
