"""Seeded synthetic inputs: corpora, query streams and probe batches.

These stand in for the paper's document sources (about 21-24 million 768-d
passage embeddings, Section 4.2.1) and query sets (questions repeated with
small variations, drawn with a Zipf skew, independent of one another, Sections
2.2 and 4.2.2).  The module only draws random numbers and normalises vectors;
it holds none of the cache's or the search's arithmetic and is the one piece of
code that both the CUDA tests and the CPU oracle's tests get their bytes from.

Recipe
  corpus   x = normalize(mu_c + 0.3 g), c uniform over the mixture components,
           mu_c ~ N(0, I_d) per component, g ~ N(0, I_d); fp32, unit norm.
  topics   T distinct corpus rows, drawn uniformly without replacement.
  stream   rank r ~ finite Zipf on 1..T with P(r) proportional to r^-s, query
           q = normalize(x_topic(r) + sigma g); draws are independent.
  probe    keys are mixture draws; a batch is half queries around random keys
           (noise sigma) and half fresh mixture draws, shuffled.

Every tensor is produced in chunks, each chunk from its own generator seeded
by (seed, stream id, chunk index), so a large corpus can be built in place on a
GPU and a small one on the CPU with the same code.  The bytes depend on the
device that draws them (CPU and CUDA generators differ); callers hand the same
bytes to both sides of a comparison.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

_STREAM_CENTRES, _STREAM_CORPUS, _STREAM_TOPICS, _STREAM_RANKS, _STREAM_NOISE, _STREAM_PROBE = range(6)


def _gen(device, seed: int, stream: int, chunk: int = 0) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1_000_003 + stream * 10_007 + chunk * 101 + 12345) % (2**63 - 1))
    return g


def _normalize_(x: torch.Tensor) -> torch.Tensor:
    return x.div_(x.norm(dim=1, keepdim=True).clamp_min_(1e-30))


def mixture_centres(n_components: int, d: int, seed: int, device="cpu") -> torch.Tensor:
    return torch.randn(n_components, d, generator=_gen(device, seed, _STREAM_CENTRES),
                       device=device, dtype=torch.float32)


def mixture_rows(n: int, centres: torch.Tensor, seed: int, stream: int = _STREAM_CORPUS,
                 chunk_rows: int = 1 << 18, out: torch.Tensor | None = None,
                 sigma: float = 0.3) -> torch.Tensor:
    """n unit-norm rows from the Gaussian mixture, written chunk by chunk into ``out``."""
    device = centres.device
    d = centres.shape[1]
    if out is None:
        out = torch.empty(n, d, device=device, dtype=torch.float32)
    for ci, r0 in enumerate(range(0, n, chunk_rows)):
        r1 = min(n, r0 + chunk_rows)
        g = _gen(device, seed, stream, ci)
        comp = torch.randint(0, centres.shape[0], (r1 - r0,), generator=g, device=device)
        x = torch.randn(r1 - r0, d, generator=g, device=device, dtype=torch.float32)
        x.mul_(sigma).add_(centres[comp])
        out[r0:r1] = _normalize_(x)
    return out


def make_corpus(N: int, d: int, n_components: int, seed: int = 0, device="cpu",
                chunk_rows: int = 1 << 18) -> torch.Tensor:
    centres = mixture_centres(n_components, d, seed, device)
    return mixture_rows(N, centres, seed, chunk_rows=chunk_rows)


def make_corpus_shard(N: int, d: int, n_components: int, seed: int, device, first: int, count: int,
                      keep_rows: torch.Tensor | None = None, chunk_rows: int = 1 << 18):
    """Rows [first, first + count) of make_corpus(N, ...) without holding the whole corpus: every
    chunk is drawn as make_corpus draws it, the shard's part is kept.  With keep_rows (int64 row
    ids of the whole corpus) the second result holds those rows too (the topics of a query
    stream may live in any shard)."""
    centres = mixture_centres(n_components, d, seed, device)
    shard = torch.empty(count, d, device=device, dtype=torch.float32)
    kept = None if keep_rows is None else torch.empty(keep_rows.numel(), d, device=device, dtype=torch.float32)
    for ci, r0 in enumerate(range(0, N, chunk_rows)):
        r1 = min(N, r0 + chunk_rows)
        a, b = max(r0, first), min(r1, first + count)
        sel = None
        if keep_rows is not None:
            sel = torch.nonzero((keep_rows >= r0) & (keep_rows < r1)).flatten()
        if a >= b and (sel is None or sel.numel() == 0):
            continue
        g = _gen(device, seed, _STREAM_CORPUS, ci)
        comp = torch.randint(0, centres.shape[0], (r1 - r0,), generator=g, device=device)
        x = torch.randn(r1 - r0, d, generator=g, device=device, dtype=torch.float32)
        x = _normalize_(x.mul_(0.3).add_(centres[comp]))
        if a < b:
            shard[a - first:b - first] = x[a - r0:b - r0]
        if sel is not None and sel.numel():
            kept[sel] = x[keep_rows[sel] - r0]
    return shard, kept


def pick_topics(N: int, T: int, seed: int = 0, device="cpu") -> torch.Tensor:
    """T distinct row indices (int64), in the order that defines the Zipf ranks."""
    assert T <= N
    g = _gen(device, seed, _STREAM_TOPICS)
    if N <= 1 << 27:
        return torch.randperm(N, generator=g, device=device)[:T].clone()
    # very large N: draw with replacement, keep the first T distinct values in draw order
    picked = torch.empty(0, dtype=torch.int64, device=device)
    while picked.numel() < T:
        cand = torch.randint(0, N, (2 * T,), generator=g, device=device)
        allv = torch.cat([picked, cand])
        uniq, inv = torch.unique(allv, return_inverse=True)
        first = torch.full((uniq.numel(),), allv.numel(), dtype=torch.int64, device=device)
        first.scatter_reduce_(0, inv, torch.arange(allv.numel(), device=device), reduce="amin")
        picked = allv[torch.sort(first).values][:T]
    return picked


def zipf_ranks(T: int, s: float, n: int, seed: int = 0, device="cpu") -> torch.Tensor:
    """n independent ranks in 0..T-1 with P(r) proportional to (r+1)^-s."""
    w = torch.arange(1, T + 1, dtype=torch.float64).pow(-s)
    cdf = torch.cumsum(w / w.sum(), 0).to(device)
    u = torch.rand(n, generator=_gen(device, seed, _STREAM_RANKS), device=device, dtype=torch.float64)
    return torch.searchsorted(cdf, u).clamp_(max=T - 1)


def noisy_copies(base_rows: torch.Tensor, sigma: float, seed: int, stream: int = _STREAM_NOISE,
                 chunk_rows: int = 1 << 16) -> torch.Tensor:
    """normalize(row + sigma g) for every given row."""
    n, d = base_rows.shape
    out = torch.empty_like(base_rows)
    for ci, r0 in enumerate(range(0, n, chunk_rows)):
        r1 = min(n, r0 + chunk_rows)
        g = torch.randn(r1 - r0, d, generator=_gen(base_rows.device, seed, stream, ci),
                        device=base_rows.device, dtype=torch.float32)
        out[r0:r1] = _normalize_(g.mul_(sigma).add_(base_rows[r0:r1]))
    return out


def make_query_stream(corpus: torch.Tensor, n_queries: int, n_topics: int, zipf_s: float,
                      sigma: float, seed: int = 0):
    """Returns (queries[n,d] fp32 unit norm, topic_rank[n] int64, topic_rows[T] int64)."""
    device = corpus.device
    topic_rows = pick_topics(corpus.shape[0], n_topics, seed, device)
    ranks = zipf_ranks(n_topics, zipf_s, n_queries, seed, device)
    q = noisy_copies(corpus[topic_rows[ranks]], sigma, seed)
    return q, ranks, topic_rows


def make_query_stream_from_topics(topic_data: torch.Tensor, n_queries: int, zipf_s: float, sigma: float,
                                  seed: int = 0) -> torch.Tensor:
    """The queries of make_query_stream when only the topics' rows are at hand: topic_data =
    corpus[pick_topics(N, T, seed)]."""
    ranks = zipf_ranks(topic_data.shape[0], zipf_s, n_queries, seed, topic_data.device)
    return noisy_copies(topic_data[ranks], sigma, seed)


def make_probe_keys(C: int, d: int, n_components: int, seed: int = 0, device="cpu"):
    centres = mixture_centres(n_components, d, seed, device)
    return mixture_rows(C, centres, seed), centres


def make_probe_batch(keys: torch.Tensor, centres: torch.Tensor, B: int, sigma: float, seed: int,
                     batch_index: int) -> torch.Tensor:
    """Half of the batch sits near random keys, half are fresh mixture draws; shuffled."""
    device = keys.device
    g = _gen(device, seed, _STREAM_PROBE, batch_index)
    n_near = B // 2
    pick = torch.randint(0, keys.shape[0], (n_near,), generator=g, device=device)
    near = noisy_copies(keys[pick], sigma, seed, stream=_STREAM_PROBE + 1 + 2 * batch_index)
    fresh = mixture_rows(B - n_near, centres, seed, stream=_STREAM_PROBE + 2 + 2 * batch_index)
    q = torch.cat([near, fresh])
    return q[torch.randperm(B, generator=g, device=device)].contiguous()


@dataclass(frozen=True)
class Config:
    """One of the benchmark workloads (sizes follow the published configurations)."""
    name: str
    N: int
    d: int
    n_components: int
    n_queries: int
    n_topics: int
    zipf_s: float
    sigma: float
    capacity: int
    policy: str
    k: int
    batch: int
    taus: tuple

    def scaled(self, **kw) -> "Config":
        return Config(**{**self.__dict__, **kw})


CONFIGS = {
    "tiny": Config("tiny", 10_000, 768, 64, 1_000, 100, 1.1, 0.02, 200, "fifo", 10, 1, (0.5,)),
    "1m": Config("1m", 1_000_000, 768, 1_024, 100_000, 2_000, 1.1, 0.02, 1_000, "lru", 10, 64,
                 (0.0, 0.25, 0.5, 1.0, 2.0)),
    "large": Config("large", 24_000_000, 768, 16_384, 200_000, 20_000, 1.0, 0.03, 10_000, "lru", 32, 256,
                    (0.0, 0.5, 1.0)),
    "lowhit": Config("lowhit", 100_000_000, 128, 65_536, 500_000, 100_000, 0.6, 0.05, 50_000, "fifo",
                     10, 1_024, (0.3,)),
}
PROBE_SIZES = (1 << 10, 1 << 14, 1 << 17, 1 << 20)


def build_workload(cfg: Config, seed: int = 0, device="cpu"):
    """(corpus, queries, ranks, topic_rows) for a configuration."""
    corpus = make_corpus(cfg.N, cfg.d, cfg.n_components, seed, device)
    q, ranks, topic_rows = make_query_stream(corpus, cfg.n_queries, cfg.n_topics, cfg.zipf_s,
                                             cfg.sigma, seed)
    return corpus, q, ranks, topic_rows
