"""ctypes binding of libspin.so: argument marshalling only.

Every step of the decode path runs in the CUDA library; this module loads it, mirrors the
structs of include/spin.h and exposes the entry points under their C names, plus a thin
`Spin` convenience class that owns the torch-allocated HBM pool.  There is no CPU fallback:
importing works without a GPU (so that the exported symbols can be checked), but any call
that needs the device fails with the library's own error.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libspin.so")

SPIN_OK = 0
STATUS_NAMES = {0: "SPIN_OK", 1: "SPIN_ERR_INVALID", 2: "SPIN_ERR_STATE", 3: "SPIN_ERR_OOM_DEVICE",
                4: "SPIN_ERR_OOM_HOST", 5: "SPIN_ERR_BUDGET", 6: "SPIN_ERR_CUDA", 7: "SPIN_ERR_TIMEOUT"}
PART_PAGE_MINMAX, PART_TOKEN_DOT, PART_CLUSTER_CENTROID, PART_PAGE_MEAN = 0, 1, 2, 3
PAGE_BYTES = 8192

EXPORTS = ["spin_required_bytes", "spin_create", "spin_destroy", "spin_request_open", "spin_reindex",
           "spin_request_close", "spin_set_budget", "spin_append_kv", "spin_append_kv_batch", "spin_decode_step",
           "spin_decode_step_append", "spin_stats", "spin_profile", "spin_profile_read", "spin_debug_dump",
           "spin_debug_read_page", "spin_debug_wait_probe", "spin_debug_link_probe", "spin_debug_launch_floor", "spin_paged_attention_static", "spin_last_error",
           "spin_version"]
KERNEL_NAMES = ["append", "score", "topk", "cache", "fetch", "attn_split", "unused"]


class SpinError(RuntimeError):
    def __init__(self, code: int, msg: str):
        super().__init__(f"{STATUS_NAMES.get(code, code)}: {msg}")
        self.code = code


class spin_config(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("device", C.c_int32), ("num_layers", C.c_int32),
                ("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("page_tokens", C.c_int32), ("max_requests", C.c_int32),
                ("max_context_tokens", C.c_int64), ("partition_kind", C.c_int32),
                ("topk", C.c_int32), ("num_clusters", C.c_int32),
                ("max_selected_pages", C.c_int32), ("max_tail_tokens", C.c_int32),
                ("lru_buckets", C.c_int32), ("segment_entries", C.c_int32),
                ("sm_scale", C.c_float), ("trace", C.c_int32), ("fetch_mode", C.c_int32),
                ("host_tables_only", C.c_int32), ("evict_exact", C.c_int32), ("resident_scoring", C.c_int32), ("reserved0", C.c_int32),
                ("offload_stage_bytes", C.c_int64),
                ("gpu_cache_pages", C.c_int64),
                ("host_pages", C.c_int64), ("hbm_pool", C.c_void_p), ("hbm_pool_bytes", C.c_size_t)]


class spin_stats_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("error_bits", C.c_uint32)] + [
        (n, C.c_uint64) for n in ("set_steps", "selected_partitions", "selected_pages", "tail_pages",
                                  "hit_pages", "miss_pages", "evicted_pages", "bypass_pages",
                                  "candidates_scored", "pcie_bytes", "hbm_bytes", "kernel_launches",
                                  "gpu_meta_bytes", "host_meta_bytes", "summary_bytes",
                                  "gpu_pages_in_use", "host_pages_in_use", "first_error_site")] + [
        ("debug_words", C.c_uint32 * 4)]


class spin_profile_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32), ("n_kernels", C.c_uint32),
                ("launches", C.c_uint64 * 8), ("ms", C.c_double * 8)]


_I32P = C.POINTER(C.c_int32)
_U32P = C.POINTER(C.c_uint32)


class spin_dump_t(C.Structure):
    _fields_ = [("struct_size", C.c_uint32),
                ("cap_selected", C.c_int32), ("cap_parts", C.c_int32), ("cap_pages", C.c_int32),
                ("cap_slots", C.c_int32), ("cap_partitions", C.c_int32), ("cap_scores", C.c_int32),
                ("n_selected", C.c_int32), ("selected", _I32P),
                ("n_parts", C.c_int32), ("parts", _I32P), ("part_state", _I32P),
                ("n_pages", C.c_int32), ("page_partition", _I32P), ("page_idx", _I32P),
                ("page_mask", _U32P), ("page_slot", _I32P),
                ("n_slots", C.c_int32), ("slot_partition", _I32P), ("slot_page_idx", _I32P),
                ("slot_ts", _I32P), ("slot_evicted_partition", _I32P),
                ("slot_evicted_page_idx", _I32P),
                ("n_partitions", C.c_int32), ("part_tokens", _I32P), ("part_resident", _I32P),
                ("n_scores", C.c_int32), ("scores", C.POINTER(C.c_float)),
                ("n_tokens", C.c_int64), ("step", C.c_int32), ("tail_pages", C.c_int32),
                ("tail_len", C.c_int32)]


_lib: Optional[C.CDLL] = None


def load() -> C.CDLL:
    """Load libspin.so (built in-tree by build.py).  Fails loudly when it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with "
                          "`python -m paper_2604_26837_b200.build` (there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    lib.spin_required_bytes.argtypes = [C.POINTER(spin_config), C.POINTER(C.c_size_t), C.POINTER(C.c_size_t)]
    lib.spin_create.argtypes = [C.POINTER(spin_config), C.POINTER(vp)]
    lib.spin_destroy.argtypes = [vp]
    lib.spin_request_open.argtypes = [vp, i64, _I32P]
    lib.spin_request_close.argtypes = [vp, i32]
    lib.spin_set_budget.argtypes = [vp, i32, i64]
    lib.spin_reindex.argtypes = [vp, i32, i32, vp]
    lib.spin_append_kv.argtypes = [vp, i32, i32, vp, vp, i64, vp, vp, vp]
    lib.spin_append_kv_batch.argtypes = [vp, i32, _I32P, i32, vp, vp, vp]
    lib.spin_decode_step.argtypes = [vp, i32, _I32P, i32, vp, vp, vp]
    lib.spin_decode_step_append.argtypes = [vp, i32, _I32P, i32, vp, vp, vp, vp, vp]
    lib.spin_stats.argtypes = [vp, C.POINTER(spin_stats_t)]
    lib.spin_profile.argtypes = [vp, i32]
    lib.spin_profile_read.argtypes = [vp, C.POINTER(spin_profile_t)]
    lib.spin_debug_dump.argtypes = [vp, i32, i32, i32, C.POINTER(spin_dump_t)]
    lib.spin_debug_read_page.argtypes = [vp, i32, i32, i32, i32, i32, i32, vp]
    lib.spin_debug_wait_probe.argtypes = [vp, i32, vp]
    lib.spin_debug_link_probe.argtypes = [vp, C.c_int64, vp]
    lib.spin_debug_launch_floor.argtypes = [vp, vp]
    lib.spin_paged_attention_static.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, C.c_float, vp, vp]
    lib.spin_last_error.argtypes = [vp]
    lib.spin_last_error.restype = C.c_char_p
    lib.spin_version.argtypes = []
    lib.spin_version.restype = C.c_char_p
    for name in EXPORTS:
        if name not in ("spin_last_error", "spin_version"):
            getattr(lib, name).restype = C.c_int
    _lib = lib
    return lib


def _ptr(x) -> Optional[int]:
    """Address of a torch tensor / numpy array / int / None."""
    try:
        return x.data_ptr()                      # torch tensor: the common case, no type tests
    except AttributeError:
        pass
    if x is None:
        return None
    if isinstance(x, int):
        return x
    if hasattr(x, "ctypes"):
        return x.ctypes.data
    raise TypeError(type(x))


def _stream_ptr(stream) -> Optional[int]:
    if stream is None:
        return None
    return stream if isinstance(stream, int) else stream.cuda_stream


def make_config(**kw) -> spin_config:
    cfg = spin_config()
    cfg.struct_size = C.sizeof(spin_config)
    cfg.head_dim, cfg.page_tokens, cfg.lru_buckets = 128, 16, 64
    for k, v in kw.items():
        if not hasattr(cfg, k):
            raise AttributeError(k)
        setattr(cfg, k, v)
    return cfg


def spin_required_bytes(cfg: spin_config):
    dev, host = C.c_size_t(0), C.c_size_t(0)
    rc = load().spin_required_bytes(C.byref(cfg), C.byref(dev), C.byref(host))
    if rc:
        raise SpinError(rc, "spin_required_bytes rejected the configuration")
    return dev.value, host.value


def spin_paged_attention_static(q, page_pool, page_ids, page_masks, n_pages, n_sets: int,
                                list_stride: int, group: int, sm_scale: float, out, stream=None):
    """Allocation-free paged attention over caller-supplied page lists (all device buffers).

    For callers that cannot allocate GPU memory and so cannot create a `Spin` context: the
    split-K scratch is an array inside the library.  Returns the status code; a request beyond
    the built-in scratch is refused (SPIN_ERR_INVALID) and explained on stderr."""
    return load().spin_paged_attention_static(_ptr(q), _ptr(page_pool), _ptr(page_ids), _ptr(page_masks),
                                              _ptr(n_pages), n_sets, list_stride, group, sm_scale,
                                              _ptr(out), _stream_ptr(stream))


class Spin:
    """One library context; methods are the C entry points with Python argument types."""

    def __init__(self, cfg: spin_config, device=None):
        import torch
        self.lib = load()
        if not torch.cuda.is_available():
            raise RuntimeError("paper_2604_26837_b200 needs a CUDA device; there is no CPU path")
        self.device = torch.device("cuda", cfg.device) if device is None else torch.device(device)
        dev_bytes, self.host_bytes = spin_required_bytes(cfg)
        # the only device allocation: one pool handed to the library
        self.pool = torch.empty(dev_bytes + 256, dtype=torch.uint8, device=self.device)
        base = (self.pool.data_ptr() + 255) // 256 * 256
        cfg.hbm_pool, cfg.hbm_pool_bytes = base, dev_bytes
        self.cfg = cfg
        self.dev_bytes = dev_bytes
        h = C.c_void_p()
        rc = self.lib.spin_create(C.byref(cfg), C.byref(h))
        if rc:
            raise SpinError(rc, "spin_create failed (see stderr)")
        self.h = h

    def _ck(self, rc: int):
        if rc:
            raise SpinError(rc, self.lib.spin_last_error(self.h).decode())

    def close(self):
        if getattr(self, "h", None):
            self.lib.spin_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def request_open(self, budget_pages_per_set: int) -> int:
        r = C.c_int32(-1)
        self._ck(self.lib.spin_request_open(self.h, budget_pages_per_set, C.byref(r)))
        return r.value

    def request_close(self, req: int):
        self._ck(self.lib.spin_request_close(self.h, req))

    def set_budget(self, req: int, budget_pages_per_set: int):
        self._ck(self.lib.spin_set_budget(self.h, req, budget_pages_per_set))

    def append_kv(self, req: int, layer: int, k, v, n_tokens: int, token_partition=None,
                  centroids=None, stream=None):
        self._ck(self.lib.spin_append_kv(self.h, req, layer, _ptr(k), _ptr(v), n_tokens,
                                         _ptr(token_partition), _ptr(centroids), _stream_ptr(stream)))

    def append_kv_batch(self, layer: int, req_ids: Sequence[int], k, v, stream=None):
        arr = (C.c_int32 * len(req_ids))(*req_ids)
        self._ck(self.lib.spin_append_kv_batch(self.h, layer, arr, len(req_ids), _ptr(k), _ptr(v),
                                               _stream_ptr(stream)))

    def decode_step(self, layer: int, req_ids: Sequence[int], q, out, stream=None):
        arr = (C.c_int32 * len(req_ids))(*req_ids)
        self._ck(self.lib.spin_decode_step(self.h, layer, arr, len(req_ids), _ptr(q), _ptr(out),
                                           _stream_ptr(stream)))

    def reindex(self, req: int, layer: int, stream=None):
        self._ck(self.lib.spin_reindex(self.h, req, layer, _stream_ptr(stream)))

    def req_array(self, req_ids: Sequence[int]):
        """The request ids as the int32 array the library takes (callers of the per-step entry
        points may build it once and pass it instead of the list)."""
        return (C.c_int32 * len(req_ids))(*req_ids)

    def decode_step_append(self, layer: int, req_ids, k_new, v_new, q, out, stream=None):
        # the per-token call: as little Python as possible before the library gets control
        arr = req_ids if isinstance(req_ids, C.Array) else (C.c_int32 * len(req_ids))(*req_ids)
        rc = self.lib.spin_decode_step_append(self.h, layer, arr, len(arr), _ptr(k_new), _ptr(v_new),
                                              _ptr(q), _ptr(out), None if stream is None else _stream_ptr(stream))
        if rc:
            self._ck(rc)

    def stats(self) -> dict:
        s = spin_stats_t()
        s.struct_size = C.sizeof(spin_stats_t)
        rc = self.lib.spin_stats(self.h, C.byref(s))
        if rc not in (0, 7):                     # SPIN_ERR_TIMEOUT still fills the counters: see "status"
            self._ck(rc)
        out = {n: getattr(s, n) for n, _ in spin_stats_t._fields_ if n not in ("struct_size", "debug_words")}
        out["debug_words"] = list(s.debug_words)
        out["status"] = rc
        return out

    def debug_launch_floor(self, stream=None):
        self._ck(self.lib.spin_debug_launch_floor(self.h, _stream_ptr(stream)))

    def debug_link_probe(self, n_pages: int, stream=None):
        self._ck(self.lib.spin_debug_link_probe(self.h, n_pages, _stream_ptr(stream)))

    def debug_wait_probe(self, max_polls: int, stream=None):
        self._ck(self.lib.spin_debug_wait_probe(self.h, max_polls, _stream_ptr(stream)))

    def profile(self, enable: bool):
        self._ck(self.lib.spin_profile(self.h, 1 if enable else 0))

    def profile_read(self) -> dict:
        """Per kernel: (launches, total ms) between CUDA events recorded on the stream."""
        p = spin_profile_t()
        p.struct_size = C.sizeof(spin_profile_t)
        self._ck(self.lib.spin_profile_read(self.h, C.byref(p)))
        return {KERNEL_NAMES[i]: (int(p.launches[i]), float(p.ms[i])) for i in range(p.n_kernels)}

    def debug_dump(self, req: int, layer: int, kv_head: int, cap_selected: int, cap_pages: int,
                   cap_slots: int, cap_partitions: int, cap_scores: int = 0) -> dict:
        import numpy as np
        d = spin_dump_t()
        d.struct_size = C.sizeof(spin_dump_t)
        bufs = {}

        def arr(name, n, dtype=np.int32, ctype=_I32P):
            a = np.zeros(max(n, 1), dtype=dtype)
            bufs[name] = a
            setattr(d, name, a.ctypes.data_as(ctype))
        d.cap_selected, d.cap_parts, d.cap_pages = cap_selected, cap_selected, cap_pages
        d.cap_slots, d.cap_partitions, d.cap_scores = cap_slots, cap_partitions, cap_scores
        arr("selected", cap_selected)
        arr("parts", cap_selected)
        arr("part_state", cap_selected)
        for n in ("page_partition", "page_idx", "page_slot"):
            arr(n, cap_pages)
        arr("page_mask", cap_pages, np.uint32, _U32P)
        for n in ("slot_partition", "slot_page_idx", "slot_ts"):
            arr(n, cap_slots)
        if self.cfg.trace:
            arr("slot_evicted_partition", cap_slots)
            arr("slot_evicted_page_idx", cap_slots)
        arr("part_tokens", cap_partitions)
        arr("part_resident", cap_partitions)
        if cap_scores:
            arr("scores", cap_scores, np.float32, C.POINTER(C.c_float))
        self._ck(self.lib.spin_debug_dump(self.h, req, layer, kv_head, C.byref(d)))
        out = dict(n_tokens=d.n_tokens, step=d.step, tail_pages=d.tail_pages, tail_len=d.tail_len)
        out["selected"] = bufs["selected"][:d.n_selected].copy()
        out["parts"] = bufs["parts"][:d.n_parts].copy()
        out["part_state"] = bufs["part_state"][:d.n_parts].copy()
        for n in ("page_partition", "page_idx", "page_slot", "page_mask"):
            out[n] = bufs[n][:d.n_pages].copy()
        for n in ("slot_partition", "slot_page_idx", "slot_ts", "slot_evicted_partition",
                  "slot_evicted_page_idx"):
            if n in bufs:
                out[n] = bufs[n][:d.n_slots].copy()
        out["part_tokens"] = bufs["part_tokens"][:d.n_partitions].copy()
        out["part_resident"] = bufs["part_resident"][:d.n_partitions].copy()
        if cap_scores:
            out["scores"] = bufs["scores"][:d.n_scores].copy()
        return out

    def debug_read_page(self, req: int, layer: int, kv_head: int, slot: int = -1,
                        partition: int = -1, page_idx: int = 0):
        import numpy as np
        buf = np.zeros(PAGE_BYTES // 2, dtype=np.uint16)
        self._ck(self.lib.spin_debug_read_page(self.h, req, layer, kv_head, slot, partition,
                                               page_idx, buf.ctypes.data))
        return buf.reshape(2, 16, 128)
