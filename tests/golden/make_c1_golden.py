"""Writes tests/golden/c1_oracle_trace.txt: the selections, misses and evictions of the tiny
configuration's 32 decode steps, computed by the CPU oracle alone.  Run from the repo root:
    python tests/golden/make_c1_golden.py
"""
import os
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)
sys.path.insert(0, os.path.join(ROOT, "tests"))

from test_oracle_pipeline import _c1_trace_lines  # noqa: E402

if __name__ == "__main__":
    lines, _ = _c1_trace_lines()
    out = os.path.join(ROOT, "tests", "golden", "c1_oracle_trace.txt")
    with open(out, "w") as f:
        f.write("# tiny configuration (1 request, GQA 4, 4096-token context, top-16 pages, 64 slots,\n"
                "# 8 buckets): per step the selected pages, the missed pages and slot:partition evicted.\n"
                "# Written by make_c1_golden.py from the CPU oracle only.\n")
        f.write("\n".join(lines) + "\n")
    print("wrote", out, len(lines), "steps")
