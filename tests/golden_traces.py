"""Reader for the hand-traced fixtures in tests/golden (see the README there)."""
import glob
import os

import numpy as np

GOLDEN_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def load_trace(path, d=16):
    params, rows = None, []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if params is None:
            params = dict(tok.split("=") for tok in line.split())
            continue
        t = line.split()
        rows.append((float(t[0]), int(t[1]), int(t[2]), int(t[3]), [int(x) for x in t[4:]]))
    k = int(params["k"])
    n_pts = int(params["corpus_points"])
    corpus = np.zeros((n_pts, d), np.float32)
    corpus[:, 0] = np.arange(n_pts)
    queries = np.zeros((len(rows), d), np.float32)
    queries[:, 0] = [r[0] for r in rows]
    preload = None
    if "preload" in params:                                   # keys bulk-loaded before the first query
        vals = [float(x) for x in params["preload"].split(",")]
        preload = np.zeros((len(vals), d), np.float32)
        preload[:, 0] = vals
    return dict(name=os.path.basename(path), policy=params["policy"], capacity=int(params["capacity"]), k=k,
                tau=float(params["tau"]), corpus=corpus, queries=queries, preload=preload,
                hit=np.array([r[1] for r in rows], np.uint8), slot=np.array([r[2] for r in rows]),
                evicted=np.array([r[3] for r in rows]), ids=np.array([r[4] for r in rows], np.int64))


def all_traces(d=16):
    return [load_trace(p, d) for p in sorted(glob.glob(os.path.join(GOLDEN_DIR, "trace_*.txt")))]


def all_load_traces(d=16):
    """Traces that start from a bulk-loaded cache (`preload=` in the header line)."""
    return [load_trace(p, d) for p in sorted(glob.glob(os.path.join(GOLDEN_DIR, "load_*.txt")))]
