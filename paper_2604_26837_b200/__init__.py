"""B200-native sparse decode step over a hierarchical paged KV cache (C-ABI library + binding).

The product is `libspin.so` (CUDA, sm_100a), declared in include/spin.h; `binding` only
marshals arguments.  Nothing here computes on the CPU.
"""
from .binding import (EXPORTS, KERNEL_NAMES, LIB_PATH, PART_CLUSTER_CENTROID, PART_PAGE_MEAN, PART_PAGE_MINMAX, PART_TOKEN_DOT,
                      Spin, SpinError, load, make_config, spin_config, spin_dump_t,
                      spin_paged_attention_static, spin_required_bytes, spin_stats_t)

__all__ = ["EXPORTS", "KERNEL_NAMES", "LIB_PATH", "PART_CLUSTER_CENTROID", "PART_PAGE_MEAN", "PART_PAGE_MINMAX", "PART_TOKEN_DOT",
           "Spin", "SpinError", "load", "make_config", "spin_config", "spin_dump_t",
           "spin_paged_attention_static", "spin_required_bytes", "spin_stats_t"]
