"""Parity at the benchmark configurations' full sizes, in the launch configuration bench.py
times (spin_decode_step_append on the whole batch): the oracle mirrors a sample of the batch's
requests -- sets are independent, so those requests must agree bit for bit (selections, cache
traces, page lists) and within tolerance (outputs) -- plus counters' invariants over the whole
batch.  Inputs are the synthetic stand-ins of `workloads`, generated on the device."""
import pytest

import workloads as W
from test_gpu_parity import run_parity

pytestmark = pytest.mark.gpu


def test_c2_llama_shaped_full_size_sampled_request():
    w = W.scaled(W.CONFIGS["c2"], steps=20)          # 8 x 32768-token contexts, 64 sets, top-128 of 2048
    r = run_parity(w, one_call=True, check_bytes=False, oracle_reqs=[3])
    assert r["stats"]["miss_pages"] > 0 and r["stats"]["evicted_pages"] == 0   # 512 slots: still filling


def test_c2_llama_shaped_full_size_softmax_scale_one():
    # the same with sm_scale = 1: logits of the outlier-channel keys are tens of units apart, the
    # softmax is sharp and outputs are of order one, so the tolerances discriminate
    w = W.scaled(W.CONFIGS["c2"], steps=6)
    r = run_parity(w, sm_scale=1.0, one_call=True, check_bytes=False, oracle_reqs=[5])
    assert r["rel_l2"] < 2e-2 and r["stats"]["miss_pages"] > 0


def test_c2_full_size_small_budget_evicts():
    w = W.scaled(W.CONFIGS["c2"], steps=24, slots_per_set=160, lru_buckets=8)
    r = run_parity(w, one_call=True, check_bytes=True, oracle_reqs=[0])
    assert r["stats"]["evicted_pages"] > 0


def test_c3_token_granular_full_size_sampled_request():
    w = W.scaled(W.CONFIGS["c3"], steps=10)          # 65536 candidate tokens per set, top-2048, cluster top-k
    r = run_parity(w, one_call=True, check_bytes=False, oracle_reqs=[1])
    assert r["stats"]["selected_partitions"] < 4 * 10 * 2048


def test_c4_cluster_granular_full_size_sampled_request():
    w = W.scaled(W.CONFIGS["c4"], steps=8, batch=4)  # 4 of the 16 requests: 131072 tokens, 1024 clusters each
    r = run_parity(w, one_call=True, check_bytes=False, oracle_reqs=[2])
    assert r["stats"]["miss_pages"] > 0


def test_c4_cluster_granular_full_size_softmax_scale_one():
    w = W.scaled(W.CONFIGS["c4"], steps=4, batch=2)
    r = run_parity(w, sm_scale=1.0, one_call=True, check_bytes=False, oracle_reqs=[1])
    assert r["rel_l2"] < 2e-2 and r["stats"]["miss_pages"] > 0


def test_c5_mixed_batch_scaled_sampled_requests():
    # the mixed-length configuration as the benchmark scales it to one box: 16 of the 64 requests,
    # 1 of the 32 layers, contexts drawn from U[8192, 262144], per-request drift, and the same
    # per-layer share of the 60 GB budget split in proportion to sequence length
    w = W.scaled(W.CONFIGS["c5"], batch=16, num_layers=1, steps=6)
    pages_per_layer = int(60e9 / 32 / 8192 * 16 / 64)
    from paper_2604_26837_b200.driver import context_sizes
    ctx = context_sizes(w)
    longest, shortest = max(range(16), key=lambda r: ctx[r]), min(range(16), key=lambda r: ctx[r])
    r = run_parity(w, one_call=True, check_bytes=False, cache_pages_per_layer=pages_per_layer,
                   oracle_reqs=sorted({longest, shortest}))
    assert r["stats"]["miss_pages"] > 0 and r["stats"]["set_steps"] == 16 * 8 * 6
