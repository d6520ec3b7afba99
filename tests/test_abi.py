"""The C-ABI library loads and exports every symbol include/spin.h declares; host-only calls
behave.  No GPU needed (no compute call is made)."""
import ctypes as C
import os
import re
import subprocess

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2604_26837_b200 import build
    build.build()
    import paper_2604_26837_b200 as P
    return P.load()


def test_every_declared_symbol_is_exported(lib):
    import paper_2604_26837_b200 as P
    header = open(os.path.join(ROOT, "include", "spin.h")).read()
    declared = set(re.findall(r"SPIN_API\s+(?:const\s+char\s*\*|int)\s*(spin_\w+)\s*\(", header))
    assert declared == set(P.EXPORTS) and len(declared) >= 12
    for name in declared:
        assert hasattr(lib, name), name
    out = subprocess.run(["nm", "-D", "--defined-only", P.LIB_PATH], capture_output=True, text=True).stdout
    exported = set(re.findall(r" T (spin_\w+)", out))
    assert declared <= exported


def test_struct_layouts_match_the_header(lib, tmp_path):
    import paper_2604_26837_b200 as P
    src = tmp_path / "sizes.c"
    src.write_text('#include "spin.h"\n#include <stdio.h>\n#include <stddef.h>\n'
                   'int main(void){printf("%zu %zu %zu %zu %zu\\n", sizeof(spin_config), sizeof(spin_stats_t),'
                   ' sizeof(spin_dump_t), offsetof(spin_config, hbm_pool), offsetof(spin_dump_t, scores));return 0;}\n')
    exe = tmp_path / "sizes"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    got = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    assert got == [C.sizeof(P.spin_config), C.sizeof(P.spin_stats_t), C.sizeof(P.spin_dump_t),
                   P.spin_config.hbm_pool.offset, P.spin_dump_t.scores.offset]


def test_required_bytes_and_argument_checks(lib):
    import paper_2604_26837_b200 as P
    cfg = P.make_config(device=0, num_layers=1, num_q_heads=32, num_kv_heads=8, max_requests=8,
                        max_context_tokens=32768 + 512, partition_kind=P.PART_PAGE_MINMAX, topk=128,
                        gpu_cache_pages=512 * 64, host_pages=64 * 2100)
    dev, host = P.spin_required_bytes(cfg)
    assert dev >= 512 * 64 * 8192 + 64 * 2100 * 512            # cache pages + min/max summaries
    assert host >= 64 * 2100 * 8192
    # metadata is small next to the KV it maps (two-level tables sized by the working set)
    assert dev < 512 * 64 * 8192 + 64 * 2100 * 512 + (64 << 20)
    for bad in (dict(head_dim=64), dict(page_tokens=8), dict(num_q_heads=24), dict(topk=0),
                dict(lru_buckets=65), dict(segment_entries=100), dict(max_requests=0)):
        cfg2 = P.make_config(device=0, num_layers=1, num_q_heads=32, num_kv_heads=8, max_requests=8,
                             max_context_tokens=4096, partition_kind=0, topk=16, gpu_cache_pages=64,
                             host_pages=4096)
        for k, v in bad.items():
            setattr(cfg2, k, v)
        with pytest.raises(P.SpinError):
            P.spin_required_bytes(cfg2)
    assert lib.spin_create(None, None) != 0
    assert lib.spin_destroy(None) != 0
    assert lib.spin_last_error(None) == b"null context"
    assert lib.spin_version().startswith(b"spin-b200")
