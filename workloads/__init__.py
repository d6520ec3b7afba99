"""Seeded synthetic inputs for the sparse decode step: workload table and generators.

This module serves both the CPU oracle and the CUDA library and therefore holds none of
the method's arithmetic (no scoring, selection, caching or attention): it only draws
keys, values, queries and cluster assignments with the shapes and distributions of the
five benchmark configurations.

Every draw is counter based: element ``i`` of stream ``(seed, tag...)`` is
``box_muller(splitmix64(key ^ i))``, so any slice can be regenerated on any device without
generating what precedes it.  Integer hashing is bit-identical on CPU and GPU; the
transcendental part of Box-Muller may differ in the last ulp between devices, so a test
generates its inputs once and hands the same bytes to both sides.

The public long-context suites the paper measures on (inputs of 16K-120K tokens) are not
available offline; these inputs stand in for them and only borrow their length ranges.
"""
from __future__ import annotations

import dataclasses
import math
from typing import Dict, List, Optional, Tuple

import torch

PART_PAGE_MINMAX = 0
PART_TOKEN_DOT = 1
PART_CLUSTER_CENTROID = 2
PART_PAGE_MEAN = 3

_M64 = (1 << 64) - 1


def _s64(x: int) -> int:
    """Python int -> two's complement signed 64-bit value (what a torch.int64 holds)."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


_GOLDEN = _s64(0x9E3779B97F4A7C15)
_MIX1 = _s64(0xBF58476D1CE4E5B9)
_MIX2 = _s64(0x94D049BB133111EB)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right of an int64 tensor."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def _splitmix64(x: torch.Tensor) -> torch.Tensor:
    z = x + _GOLDEN
    z = (z ^ _lsr(z, 30)) * _MIX1
    z = (z ^ _lsr(z, 27)) * _MIX2
    return z ^ _lsr(z, 31)


def _py_splitmix64(x: int) -> int:
    z = (x + 0x9E3779B97F4A7C15) & _M64
    z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
    z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, *tags: int) -> int:
    """Fold a seed and integer tags into one 64-bit stream key."""
    k = _py_splitmix64(seed & _M64)
    for t in tags:
        k = _py_splitmix64(k ^ ((t + 0x632BE59BD9B4E019) & _M64))
    return k


def raw_bits(key: int, n: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n 64-bit hashes (as int64) of counters offset..offset+n-1 under `key`."""
    idx = torch.arange(offset, offset + n, dtype=torch.int64, device=device)
    return _splitmix64(idx * _MIX2 ^ _s64(key))


def normal(key: int, n: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n draws of N(0,1) in fp32 (Box-Muller on two 24-bit uniforms of one hash)."""
    out = torch.empty(n, dtype=torch.float32, device=device)
    chunk = 1 << 26
    for s in range(0, n, chunk):
        m = min(chunk, n - s)
        b = raw_bits(key, m, device, offset + s)
        u1 = ((_lsr(b, 40) & 0xFFFFFF) + 1).to(torch.float32) * (1.0 / 16777216.0)
        u2 = (_lsr(b, 16) & 0xFFFFFF).to(torch.float32) * (1.0 / 16777216.0)
        out[s:s + m] = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    return out


def uniform_int(key: int, n: int, high: int, device="cpu", offset: int = 0) -> torch.Tensor:
    """n integers uniform in [0, high) (int64)."""
    b = raw_bits(key, n, device, offset)
    return (_lsr(b, 11) % high)


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes, selection rule, cache budget, input recipe)."""
    name: str
    seed: int
    batch: int
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    page_tokens: int
    context: int                 # prefill tokens per request (or the upper bound if ctx_range)
    partition_kind: int
    topk: int                    # partitions (pages / clusters) or tokens (PART_TOKEN_DOT)
    slots_per_set: int           # HBM budget of one (request, layer, kv-head) set, in pages
    lru_buckets: int
    steps: int
    drift: float                 # sigma of the per-step query drift
    kv_recipe: str               # "normal" | "outlier" | "page_centre" | "mixture" | "tied"
    num_clusters: int = 0
    cluster_sd: float = 0.3
    outlier_channels: int = 0
    outlier_scale: float = 8.0
    centre_sd: float = 0.5
    ctx_range: Optional[Tuple[int, int]] = None      # per-request context drawn uniformly
    drift_choices: Optional[Tuple[float, ...]] = None  # per-request drift drawn from these
    max_partition_pages: int = 1
    tie_period: int = 0                              # "tied": token t carries the key of token t % tie_period
    zero_run: Optional[Tuple[int, int]] = None       # "tied": tokens [a, b) have all-zero keys
    tied_centroid_period: int = 0                    # > 0: cluster c carries the centroid of cluster c % period

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    def request_context(self, req: int) -> int:
        if self.ctx_range is None:
            return self.context
        lo, hi = self.ctx_range
        r = _py_splitmix64(stream_key(self.seed, 91, req))
        return lo + r % (hi - lo + 1)

    def request_drift(self, req: int) -> float:
        if self.drift_choices is None:
            return self.drift
        r = _py_splitmix64(stream_key(self.seed, 92, req))
        return self.drift_choices[r % len(self.drift_choices)]


def _mk(**kw) -> Workload:
    return Workload(**kw)


# Names follow the benchmark list: c1 is the tiny case, c2 the Llama-3-8B-shaped one, ...
CONFIGS: Dict[str, Workload] = {
    "c1": _mk(name="c1", seed=20260427, batch=1, num_layers=1, num_q_heads=4, num_kv_heads=1,
              head_dim=128, page_tokens=16, context=4096, partition_kind=PART_PAGE_MINMAX,
              topk=16, slots_per_set=64, lru_buckets=8, steps=32, drift=0.1,
              kv_recipe="normal"),
    "c2": _mk(name="c2", seed=20260428, batch=8, num_layers=1, num_q_heads=32, num_kv_heads=8,
              head_dim=128, page_tokens=16, context=32768, partition_kind=PART_PAGE_MINMAX,
              topk=128, slots_per_set=512, lru_buckets=64, steps=256, drift=0.05,
              kv_recipe="outlier", outlier_channels=4, outlier_scale=8.0),
    "c3": _mk(name="c3", seed=20260429, batch=4, num_layers=1, num_q_heads=4, num_kv_heads=1,
              head_dim=128, page_tokens=16, context=65536, partition_kind=PART_TOKEN_DOT,
              topk=2048, slots_per_set=819, lru_buckets=64, steps=128, drift=0.05,
              kv_recipe="page_centre", centre_sd=0.5),
    "c4": _mk(name="c4", seed=20260430, batch=16, num_layers=1, num_q_heads=32, num_kv_heads=8,
              head_dim=128, page_tokens=16, context=131072,
              partition_kind=PART_CLUSTER_CENTROID, topk=64, slots_per_set=868,
              lru_buckets=64, steps=128, drift=0.05, kv_recipe="mixture", num_clusters=1024,
              cluster_sd=0.3, max_partition_pages=16),
    "c5": _mk(name="c5", seed=20260431, batch=64, num_layers=32, num_q_heads=32,
              num_kv_heads=8, head_dim=128, page_tokens=16, context=262144,
              partition_kind=PART_PAGE_MINMAX, topk=256, slots_per_set=0, lru_buckets=64,
              steps=64, drift=0.1, kv_recipe="normal", ctx_range=(8192, 262144),
              drift_choices=(0.01, 0.1, 0.5)),
}


def scaled(w: Workload, **kw) -> Workload:
    """A smaller (or otherwise edited) copy of a workload, for tests."""
    return dataclasses.replace(w, **kw)


def _bf16(x: torch.Tensor) -> torch.Tensor:
    return x.to(torch.bfloat16)


def outlier_channels(w: Workload, layer: int, head: int) -> List[int]:
    """The channels of one kv head whose keys are scaled up (same for every request)."""
    chans: List[int] = []
    i = 0
    while len(chans) < w.outlier_channels:
        c = _py_splitmix64(stream_key(w.seed, 93, layer, head, i)) % w.head_dim
        if c not in chans:
            chans.append(c)
        i += 1
    return sorted(chans)


_SCALE_CACHE: dict = {}


def _outlier_scale(w: Workload, layer: int, device) -> torch.Tensor:
    """fp32 [num_kv_heads][head_dim]: outlier_scale on the outlier channels, 1 elsewhere."""
    key = (w.seed, w.num_kv_heads, w.head_dim, w.outlier_channels, w.outlier_scale, layer, str(device))
    if key not in _SCALE_CACHE:
        s = torch.ones(w.num_kv_heads, w.head_dim, dtype=torch.float32)
        for h in range(w.num_kv_heads):
            for c in outlier_channels(w, layer, h):
                s[h, c] = w.outlier_scale
        _SCALE_CACHE[key] = s.to(device)
    return _SCALE_CACHE[key]


def centroids(w: Workload, req: int, layer: int, device="cpu") -> torch.Tensor:
    """Mixture centroids of one request: bf16 [num_clusters][num_kv_heads][head_dim]."""
    n = w.num_clusters * w.num_kv_heads * w.head_dim
    c = normal(stream_key(w.seed, 3, req, layer), n, device).view(w.num_clusters, w.num_kv_heads, w.head_dim)
    if w.tied_centroid_period > 0:
        c = c[torch.arange(w.num_clusters, device=device) % w.tied_centroid_period]
    return _bf16(c)


def cluster_assignment(w: Workload, req: int, layer: int, n_tokens: int, device="cpu",
                       first_token: int = 0) -> torch.Tensor:
    """Cluster id of every (token, kv head): int32 [n_tokens][num_kv_heads]."""
    a = uniform_int(stream_key(w.seed, 4, req, layer), n_tokens * w.num_kv_heads,
                    w.num_clusters, device, first_token * w.num_kv_heads)
    return a.to(torch.int32).view(n_tokens, w.num_kv_heads)


def kv_tokens(w: Workload, req: int, layer: int, first_token: int, n_tokens: int,
              device="cpu") -> Tuple[torch.Tensor, torch.Tensor]:
    """Keys and values of tokens [first_token, first_token+n_tokens) of one request/layer.

    Returns bf16 tensors shaped [n_tokens][num_kv_heads][head_dim].  Prefill and decode
    tokens come from the same stream, so appended tokens follow the context's distribution.
    """
    H, d = w.num_kv_heads, w.head_dim
    row = H * d
    zk = normal(stream_key(w.seed, 1, req, layer), n_tokens * row, device,
                first_token * row).view(n_tokens, H, d)
    zv = normal(stream_key(w.seed, 2, req, layer), n_tokens * row, device,
                first_token * row).view(n_tokens, H, d)
    if w.kv_recipe == "normal":
        k = zk
    elif w.kv_recipe == "outlier":
        k = zk * _outlier_scale(w, layer, device)
    elif w.kv_recipe == "page_centre":
        T = w.page_tokens
        p0 = first_token // T
        p1 = (first_token + n_tokens - 1) // T + 1
        cen = normal(stream_key(w.seed, 5, req, layer), (p1 - p0) * row, device,
                     p0 * row).view(p1 - p0, H, d)
        tok = torch.arange(first_token, first_token + n_tokens, device=device)
        k = cen[(tok // T - p0)] + w.centre_sd * zk
    elif w.kv_recipe == "mixture":
        cen = centroids(w, req, layer, device).to(torch.float32)          # [C][H][d]
        a = cluster_assignment(w, req, layer, n_tokens, device, first_token).long()
        hh = torch.arange(H, device=device).view(1, H).expand(n_tokens, H)
        k = cen[a, hh] + w.cluster_sd * zk
    elif w.kv_recipe == "tied":
        # duplicated keys: the key rows repeat with period `tie_period` tokens (a multiple of the
        # page size makes whole pages repeat), and a run of tokens has all-zero keys; values stay
        # distinct.  Candidates built from equal keys have equal summaries, whatever the rule.
        tok = torch.arange(first_token, first_token + n_tokens, device=device)
        src = normal(stream_key(w.seed, 1, req, layer), w.tie_period * row, device, 0).view(w.tie_period, H, d)
        k = src[tok % w.tie_period]
        if w.zero_run is not None:
            k = torch.where(((tok >= w.zero_run[0]) & (tok < w.zero_run[1])).view(-1, 1, 1), torch.zeros_like(k), k)
    else:
        raise ValueError(w.kv_recipe)
    return _bf16(k), _bf16(zv)


class QueryStream:
    """Drifting unit-norm queries of one request/layer: q_t = normalize(q_{t-1} + s*N(0,1))."""

    def __init__(self, w: Workload, req: int, layer: int, device="cpu"):
        self.w, self.req, self.layer, self.device = w, req, layer, device
        self.sigma = w.request_drift(req)
        self.t = 0
        self.n = w.num_q_heads * w.head_dim
        z = normal(stream_key(w.seed, 6, req, layer, 0), self.n, device)
        self.q = self._normalize(z.view(w.num_q_heads, w.head_dim))

    @staticmethod
    def _normalize(x: torch.Tensor) -> torch.Tensor:
        return x / torch.linalg.vector_norm(x, dim=-1, keepdim=True)

    def next(self) -> torch.Tensor:
        """Query of the next decode step: bf16 [num_q_heads][head_dim]."""
        if self.t > 0:
            z = normal(stream_key(self.w.seed, 6, self.req, self.layer, self.t), self.n,
                       self.device).view_as(self.q)
            self.q = self._normalize(self.q + self.sigma * z)
        self.t += 1
        return _bf16(self.q)


def to_bits(x: torch.Tensor):
    """bf16 tensor -> numpy uint16 array of its bit patterns (the oracle's input format)."""
    import numpy as np
    return x.detach().cpu().contiguous().view(torch.int16).numpy().view(np.uint16)
