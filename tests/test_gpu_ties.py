"""Parity on inputs whose candidate scores are genuinely tied (duplicated keys, all-zero keys).

Select must order equal scores by the lower candidate index (the total order the oracle's
stable sort defines), so on these inputs the threshold bin of the radix select holds ties that
straddle the k-th place, all candidates can be equal, equal keys can fall into different CTAs'
slices of the cluster top-k, and products with zero keys give -0.0 that must rank as +0.0.
Everything is compared bit for bit with the oracle, as in test_gpu_parity.
"""
import pytest

import workloads as W
from test_gpu_parity import _wl, run_parity

pytestmark = pytest.mark.gpu


def _tied(kind, **kw):
    base = dict(kv_recipe="tied", num_layers=1, drift=0.3, lru_buckets=4)
    base.update(kw)
    return _wl(kind, **base)


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_PAGE_MEAN])
def test_pages_repeat_with_period_seven(kind):
    # page j carries the keys of page j % 7: seven distinct scores over 60 pages, so the k-th
    # place always falls inside a group of 8-9 equal scores
    w = _tied(kind, context=16 * 60 + 3, tie_period=16 * 7, topk=12, slots_per_set=20, steps=24)
    r = run_parity(w, one_call=True)
    assert r["tied_at_k"] == 2 * 2 * 24                   # every set, every step


def test_pages_repeat_and_a_run_of_zero_keys_scores_exactly_zero():
    # pages 10..29 hold all-zero keys: their score is +0.0 whatever the query's signs (a sum of
    # -0.0 products must not rank below +0.0), tied with one another; the other 30 pages score
    # above zero (the bound of a page of varied keys is positive), so top-36 ends six pages into
    # the zero group; GQA group 4 and 8
    for hq in (8, 16):
        w = _tied(W.PART_PAGE_MINMAX, context=16 * 50 + 9, tie_period=16 * 11, zero_run=(160, 480), topk=36,
                  slots_per_set=48, steps=16, num_q_heads=hq, num_kv_heads=2)
        r = run_parity(w, one_call=True)
        assert r["tied_at_k"] == 2 * 2 * 16


@pytest.mark.parametrize("kind", [W.PART_PAGE_MINMAX, W.PART_TOKEN_DOT])
def test_all_candidates_equal(kind):
    # every key row is the same row: all scores equal, the selection is the first k candidates
    w = _tied(kind, context=16 * 40 + 5, tie_period=1, topk=9 if kind == W.PART_PAGE_MINMAX else 70,
              slots_per_set=12, steps=20)
    r = run_parity(w, one_call=True)
    assert r["tied_at_k"] == 2 * 2 * 20


def test_all_keys_zero():
    # every score is exactly zero (products of either sign of zero)
    w = _tied(W.PART_TOKEN_DOT, context=16 * 30, tie_period=5, zero_run=(0, 1 << 30), topk=50, slots_per_set=10, steps=8)
    r = run_parity(w, one_call=True)
    assert r["tied_at_k"] == 2 * 2 * 8


def test_token_rows_repeat_inside_one_cta():
    # token granularity, 960 candidate keys with period 37: ties in the shared-memory select
    w = _tied(W.PART_TOKEN_DOT, context=16 * 60 + 2, tie_period=37, topk=100, slots_per_set=30, steps=20,
              num_q_heads=4, num_kv_heads=1)
    r = run_parity(w, one_call=True)
    assert r["tied_at_k"] == 2 * 20


def test_token_rows_repeat_across_the_slices_of_the_cluster_top_k():
    # 20800 candidate keys per set (one thread-block cluster per set, four slices of 5200 keys)
    # with period 1000: each distinct score appears 20-21 times, spread over all four slices;
    # top-300 ends inside such a group.  Then the same with every key equal.
    w = _tied(W.PART_TOKEN_DOT, context=16 * 1300 + 5, tie_period=1000, topk=300, slots_per_set=120, steps=12,
              batch=2, num_q_heads=4, num_kv_heads=2, lru_buckets=8)
    r = run_parity(w, check_bytes=False, one_call=True)
    assert r["tied_at_k"] == 2 * 2 * 12
    w = _tied(W.PART_TOKEN_DOT, context=16 * 1300 + 5, tie_period=1, topk=300, slots_per_set=40, steps=6,
              batch=1, num_q_heads=4, num_kv_heads=2, lru_buckets=8)
    r = run_parity(w, check_bytes=False, one_call=True)
    assert r["tied_at_k"] == 2 * 6
    # groups of 520 equal keys (period 40): larger than what the select ranks directly, so the
    # threshold key is decided digit by digit to its last bit, and the k-th place falls inside a group
    w = _tied(W.PART_TOKEN_DOT, context=16 * 1300 + 5, tie_period=40, topk=300, slots_per_set=60, steps=8,
              batch=1, num_q_heads=4, num_kv_heads=2, lru_buckets=8)
    r = run_parity(w, check_bytes=False, one_call=True)
    assert r["tied_at_k"] == 2 * 8


def test_pages_repeat_across_the_slices_of_the_cluster_top_k():
    # page granularity through the cluster kernel: 16500 candidate pages per set whose keys repeat
    # with a period of 7 pages (2357 equal bounds per group, spread over all slices)
    w = _tied(W.PART_PAGE_MINMAX, context=16 * 16500 + 3, tie_period=16 * 7, topk=64, slots_per_set=100, steps=6,
              batch=1, num_layers=1, num_q_heads=2, num_kv_heads=1, lru_buckets=8)
    r = run_parity(w, check_bytes=False, one_call=True)
    assert r["tied_at_k"] == 6


def test_clusters_with_equal_centroids():
    # cluster granularity: the centroids repeat with period 5, so q . centroid ties across clusters
    w = _tied(W.PART_CLUSTER_CENTROID, context=16 * 40 + 3, tie_period=64, num_clusters=30, topk=7,
              slots_per_set=40, steps=16, max_partition_pages=8, tied_centroid_period=5)
    r = run_parity(w, one_call=True)
    assert r["tied_at_k"] == 2 * 2 * 16
