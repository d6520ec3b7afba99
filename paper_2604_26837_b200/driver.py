"""Synthetic driver: feeds a `workloads.Workload` through the library, the way a serving
engine's attention layer would (prefill appends, then per decode step one appended token and
one decode call per layer).  Marshalling and input generation only; it never computes any
stage of the path itself and knows nothing about the CPU oracle.
"""
from __future__ import annotations

from typing import List, Optional

import torch

import workloads as W

from . import binding as B


def context_sizes(w: W.Workload):
    ctx = [w.request_context(r) for r in range(w.batch)]
    return ctx


def request_budgets(w: W.Workload, cache_pages_per_layer: int) -> List[int]:
    """Per-request slots per set when the workload gives a total instead of a fixed budget:
    every set first gets its mandatory pages min(top-k, its pages); what is left of the layer's
    cache is shared in proportion to sequence length and capped at the set's page count
    (Section 5.3, buffer elasticity: reclaim / grant in proportion to sequence length)."""
    T = w.page_tokens
    ctx = context_sizes(w)
    pages = [(c + w.steps + T - 1) // T for c in ctx]
    mandatory = [min(w.topk, p) for p in pages]
    left = cache_pages_per_layer // w.num_kv_heads - sum(mandatory)
    total = sum(pages)
    out = []
    for m, p in zip(mandatory, pages):
        extra = max(0, left) * p // max(total, 1)
        out.append(min(p, m + extra))
    return out


class SpinRun:
    """A library context sized for one workload, plus the per-step call sequence."""

    def __init__(self, w: W.Workload, device="cuda:0", trace=False, sm_scale=0.0,
                 slots_per_set=None, segment_entries=0, fetch_mode=0, host_tables_only=0,
                 cache_pages_per_layer=None, spare_cache_pages=0, evict_exact=0, offload_stage_bytes=0, resident_scoring=0):
        self.w = w
        self.device = torch.device(device)
        T = w.page_tokens
        ctx = context_sizes(w)
        sets_per_req = w.num_layers * w.num_kv_heads
        self.slots = w.slots_per_set if slots_per_set is None else slots_per_set
        # one budget per request (all its sets get it); a per-layer total switches to the dynamic split
        self.budgets = ([self.slots] * w.batch if cache_pages_per_layer is None
                        else request_budgets(w, cache_pages_per_layer))
        cluster = w.partition_kind == W.PART_CLUSTER_CENTROID
        pages_per_set = [(c + w.steps + T - 1) // T + 2 for c in ctx]
        if cluster:
            pages_per_set = [p + w.num_clusters for p in pages_per_set]
        host_pages = sum(pages_per_set) * sets_per_req
        cfg = B.make_config(
            device=self.device.index or 0, num_layers=w.num_layers, num_q_heads=w.num_q_heads,
            num_kv_heads=w.num_kv_heads, max_requests=w.batch,
            max_context_tokens=max(ctx) + w.steps + T, partition_kind=w.partition_kind,
            topk=w.topk, num_clusters=w.num_clusters if cluster else 0,
            max_selected_pages=(w.topk * w.max_partition_pages if cluster else 0),
            max_tail_tokens=(w.steps + T if cluster else 0), lru_buckets=w.lru_buckets,
            segment_entries=segment_entries, sm_scale=sm_scale, trace=1 if trace else 0, fetch_mode=fetch_mode, host_tables_only=host_tables_only,
            evict_exact=evict_exact, offload_stage_bytes=offload_stage_bytes, resident_scoring=resident_scoring, gpu_cache_pages=sum(self.budgets) * sets_per_req + spare_cache_pages, host_pages=host_pages)
        self.spin = B.Spin(cfg, self.device)
        self.reqs: List[int] = [self.spin.request_open(bud) for bud in self.budgets]
        self._req_arr = self.spin.req_array(self.reqs)
        self.ctx = ctx
        self.step_no = 0

    # -- inputs (synthetic, generated on the device) ------------------------------------
    def gen_prefill(self, r: int, layer: int):
        w = self.w
        k, v = W.kv_tokens(w, r, layer, 0, self.ctx[r], self.device)
        if w.partition_kind == W.PART_CLUSTER_CENTROID:
            tp = W.cluster_assignment(w, r, layer, self.ctx[r], self.device).contiguous()
            cen = W.centroids(w, r, layer, self.device).contiguous()
            return k.contiguous(), v.contiguous(), tp, cen
        return k.contiguous(), v.contiguous(), None, None

    def gen_step_tokens(self, layer: int, step: int):
        ks, vs = [], []
        for r in range(self.w.batch):
            k, v = W.kv_tokens(self.w, r, layer, self.ctx[r] + step, 1, self.device)
            ks.append(k)
            vs.append(v)
        return torch.cat(ks).contiguous(), torch.cat(vs).contiguous()      # [B][Hkv][d]

    # -- calls -----------------------------------------------------------------------------
    def prefill(self, r: int, layer: int, k, v, tp=None, cen=None, stream=None):
        self.spin.append_kv(self.reqs[r], layer, k, v, k.shape[0], tp, cen, stream)

    def append(self, layer: int, k_new, v_new, stream=None):
        self.spin.append_kv_batch(layer, self.reqs, k_new, v_new, stream)

    def decode(self, layer: int, q, out, stream=None):
        self.spin.decode_step(layer, self.reqs, q, out, stream)

    def step(self, layer: int, k_new, v_new, q, out, stream=None):
        """Append one token per request and decode, in one library call."""
        self.spin.decode_step_append(layer, self._req_arr, k_new, v_new, q, out, stream)

    def reindex(self, r: int, layer: int, stream=None):
        """Fold request r's full tail pages into its clusters (cluster granularity)."""
        self.spin.reindex(self.reqs[r], layer, stream)

    def set_budget(self, r: int, slots: int):
        """Resize the GPU slots of every set of request r (buffer elasticity)."""
        self.spin.set_budget(self.reqs[r], slots)
        self.budgets[r] = slots

    def close(self):
        self.spin.close()
