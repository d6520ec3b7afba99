"""The offline-optimal cache replay used for the ideal envelope (Section 3.1), against brute force."""
import itertools

import numpy as np

from paper_2604_26837_b200.envelope import belady_miss_pages, eq3_tpot


def brute_min_misses(trace, capacity):
    """Exhaustive search over which partitions to keep after every step (unit-size partitions)."""
    best = [10 ** 9]

    def go(t, cache, misses):
        if misses >= best[0]:
            return
        if t == len(trace):
            best[0] = misses
            return
        sel = set(trace[t])
        m = len(sel - cache)
        pool = cache | sel
        keep_n = min(capacity, len(pool))
        # the selected ones that fit must be kept (they are in use); choose the rest freely
        must = sel if len(sel) <= capacity else set()
        rest = sorted(pool - must)
        for extra in itertools.combinations(rest, max(0, keep_n - len(must))):
            go(t + 1, must | set(extra), misses + m)
    go(0, set(), 0)
    return best[0]


def test_belady_matches_exhaustive_search_on_tiny_traces():
    rng = np.random.default_rng(3)
    for trial in range(60):
        P, cap, T, k = int(rng.integers(4, 7)), int(rng.integers(2, 5)), int(rng.integers(3, 7)), 2
        trace = [sorted(set(int(x) for x in rng.integers(0, P, size=k))) for _ in range(T)]
        if max(len(s) for s in trace) > cap:
            continue
        got = belady_miss_pages(trace, {}, cap)
        assert got == brute_min_misses(trace, cap), (trace, cap)


def test_belady_never_worse_than_any_online_policy_and_counts_compulsory_misses():
    trace = [[0, 1], [1, 2], [0, 1], [3, 4], [0, 1]]
    assert belady_miss_pages(trace, {}, 100) == 5            # infinite cache: compulsory only
    assert belady_miss_pages(trace, {}, 2) == 2 + 1 + 1 + 2 + 2
    assert belady_miss_pages(trace, {p: 2 for p in range(5)}, 100) == 10


def test_eq3_terms():
    # 64 MB of summaries + 66 MB of selected KV at 6.5 TB/s, 10% of the KV over a 50 GB/s link
    t = eq3_tpot(64e6, 66e6, 0.1, 6.5e12, 50e9)
    assert abs(t - (130e6 / 6.5e12 + 6.6e6 / 50e9)) < 1e-12
