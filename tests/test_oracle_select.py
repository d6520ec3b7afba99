"""Pins for the oracle's Select stage (score + top-k).  CPU only."""
import numpy as np
import pytest

from oracle import spin_oracle as O

F32 = np.float32


def _rand_bf16(rng, shape, scale=1.0):
    x = (rng.standard_normal(shape) * scale).astype(np.float32)
    bits = (x.view(np.uint32) >> 16).astype(np.uint16)          # truncate: still valid bf16
    return bits


def test_canonical_sum_order_is_the_stated_tree():
    # Values chosen so that every other plausible order gives a different fp32 result.
    # Block 0 = [2^24, 1, 1, 1, 1, 1, 1, 1]: left to right each "+1" is absorbed
    # (ties-to-even at 2^24) -> 2^24; a pairwise order inside the block would give 2^24+8.
    d = 128
    t = np.zeros(d, dtype=F32)
    t[0] = 2.0 ** 24
    t[1:8] = 1.0
    # Blocks 1..3 each sum to 1 (a single 1.0): tree = ((b0+b1) + (b2+b3)) = 2^24 + 2,
    # whereas a left-to-right pass over block sums gives 2^24 (each +1 absorbed).
    t[8] = 1.0
    t[16] = 1.0
    t[24] = 1.0
    assert float(O.canonical_sum(t)) == 2.0 ** 24 + 2.0
    # A term in the far half joins at the last tree level: (2^24+2) + 1 -> ties-to-even
    # gives 2^24+4?  (2^24+3 is not representable; neighbours 2^24+2 (even mantissa) and
    # 2^24+4: spacing is 2, 2^24+3 is halfway -> even mantissa = 2^24+4.)
    t[64] = 1.0
    assert float(O.canonical_sum(t)) == 2.0 ** 24 + 4.0


def test_canonical_sum_exact_on_small_integers():
    rng = np.random.default_rng(1)
    t = rng.integers(-1000, 1000, size=(50, 128)).astype(F32)
    assert np.array_equal(O.canonical_sum(t), t.astype(np.int64).sum(axis=1).astype(F32))


@pytest.mark.parametrize("G", [1, 4])
def test_page_size_one_minmax_equals_dot_bitwise(G):
    rng = np.random.default_rng(2)
    q = O.bf16_to_f32(_rand_bf16(rng, (G, 128)))
    k = O.bf16_to_f32(_rand_bf16(rng, (300, 128)))
    a = O.score_minmax(q, k, k)
    b = O.score_dot(q, k)
    assert np.array_equal(a.view(np.uint32), b.view(np.uint32))


def test_minmax_score_bounds_every_key_and_matches_fp64():
    rng = np.random.default_rng(3)
    G, P, T, d = 4, 40, 16, 128
    q = O.bf16_to_f32(_rand_bf16(rng, (G, d)))
    keys = O.bf16_to_f32(_rand_bf16(rng, (P, T, d), scale=2.0))
    smin, smax = keys.min(axis=1), keys.max(axis=1)
    s = O.score_minmax(q, smin, smax).astype(np.float64)
    q64, k64 = q.astype(np.float64), keys.astype(np.float64)
    exact = np.einsum("gd,ptd->pt", q64, k64)                  # sum over heads of q_g.k
    assert (exact <= s[:, None] + 1e-3).all()
    ref = np.maximum(q64[:, None, :] * smin[None], q64[:, None, :] * smax[None]).sum(axis=(0, 2))
    assert np.allclose(s, ref, rtol=1e-5, atol=1e-4)
    # the bound is tight for a page made of one repeated key
    one = np.repeat(keys[:, :1], T, axis=1)
    s1 = O.score_minmax(q, one.min(axis=1), one.max(axis=1)).astype(np.float64)
    assert np.allclose(s1, np.einsum("gd,pd->p", q64, one[:, 0].astype(np.float64)),
                       rtol=1e-5, atol=1e-4)


def test_dot_score_matches_fp64_and_group_sum():
    rng = np.random.default_rng(4)
    q = O.bf16_to_f32(_rand_bf16(rng, (4, 128)))
    k = O.bf16_to_f32(_rand_bf16(rng, (500, 128)))
    s = O.score_dot(q, k)
    ref = k.astype(np.float64) @ q.astype(np.float64).sum(axis=0)
    assert np.allclose(s, ref, rtol=1e-5, atol=1e-4)


def test_group_heads_are_added_in_ascending_order():
    # per-head scores 2^24, 1, 1, -2^24 (one non-zero channel each, exact in bf16): ascending
    # order gives ((2^24 + 1) + 1) + -2^24 = 0 in fp32 (each +1 is lost to rounding), the reverse
    # order gives ((-2^24 + 1) + 1) + 2^24 = 2, a pairwise tree gives 0 + ... = different again
    q = np.zeros((4, 128), dtype=F32)
    q[0, 0], q[1, 0], q[2, 0], q[3, 0] = 2.0 ** 24, 1.0, 1.0, -(2.0 ** 24)
    k = np.zeros((2, 128), dtype=F32)
    k[0, 0] = 1.0
    s = O.score_dot(q, k)
    assert float(s[0]) == 0.0 and float(s[1]) == 0.0
    s_rev = O.score_dot(q[::-1].copy(), k)
    assert float(s_rev[0]) == 2.0
    lo, hi = np.zeros((2, 128), dtype=F32), np.zeros((2, 128), dtype=F32)
    lo[0, 0] = hi[0, 0] = 1.0
    assert float(O.score_minmax(q, lo, hi)[0]) == 0.0 and float(O.score_minmax(q[::-1].copy(), lo, hi)[0]) == 2.0


def test_negative_zero_is_canonicalised():
    q = np.full((1, 128), -1.0, dtype=F32)
    k = np.zeros((3, 128), dtype=F32)
    s = O.score_dot(q, k)                                       # -1 * 0 = -0.0 everywhere
    assert np.array_equal(s.view(np.uint32), np.zeros(3, dtype=np.uint32))


def _brute_topk(scores, k):
    idx = sorted(range(len(scores)), key=lambda i: (-float(scores[i]), i))
    return sorted(idx[:min(k, len(scores))])


def test_topk_against_brute_force_with_ties():
    rng = np.random.default_rng(5)
    for trial in range(200):
        n = int(rng.integers(0, 60))
        k = int(rng.integers(0, 70))
        scores = rng.integers(-3, 4, size=n).astype(F32)        # heavy ties
        if trial % 3 == 0 and n:
            scores[rng.integers(0, n)] = np.inf if trial % 2 else -np.inf
        got = O.topk_select(scores, k)
        assert list(got) == _brute_topk(scores, k)


def test_topk_tie_goes_to_lower_index_and_zero_signs_tie():
    s = np.array([1.0, 2.0, 2.0, 2.0, 0.5], dtype=F32)
    assert list(O.topk_select(s, 2)) == [1, 2]
    s = np.array([-0.0, 0.0, -1.0], dtype=F32)
    assert list(O.topk_select(s, 1)) == [0]
    assert list(O.topk_select(s, 10)) == [0, 1, 2]


def _mean_set(keys_bits):
    """An oracle set of the landmark kind holding one indexed page made of `keys_bits` (16 rows)."""
    cfg = O.OracleConfig(1, 1, 1, partition_kind=O.PART_PAGE_MEAN)
    st = O.OracleSet(cfg, 4)
    st.append_tokens(keys_bits, keys_bits)
    st.append_tokens(keys_bits[:1], keys_bits[:1])          # first token of the next page indexes it
    return st


def test_mean_summary_special_cases_and_rounding():
    rng = np.random.default_rng(9)
    one = _rand_bf16(rng, (1, 128))
    st = _mean_set(np.repeat(one, 16, axis=0))              # 16 equal keys: the mean is the key
    assert np.array_equal(st.sum_vec[0], O.bf16_to_f32(one[0]))
    pair = np.concatenate([one, one ^ np.uint16(0x8000)] * 8)   # x, -x, x, -x ...: the mean is 0
    assert np.array_equal(_mean_set(pair).sum_vec[0], np.zeros(128, dtype=F32))
    keys = _rand_bf16(rng, (16, 128), scale=3.0)
    got = _mean_set(keys).sum_vec[0]
    exact = O.bf16_to_f32(keys).astype(np.float64).mean(axis=0)
    assert np.array_equal(got, O.f32_to_bf16_f32(got))      # a bf16 value
    # within half a bf16 ulp of the exact mean (plus the fp32 summation error, far smaller)
    assert (np.abs(got - exact) <= np.abs(exact) * 2.0 ** -8 + 1e-30).all()
    # small integers: exact arithmetic, so the value is fixed whatever the order
    ints = rng.integers(-8, 8, size=(16, 128)).astype(np.float32)
    ibits = (ints.view(np.uint32) >> 16).astype(np.uint16)
    assert np.array_equal(_mean_set(ibits).sum_vec[0], O.f32_to_bf16_f32((ints.sum(axis=0) / 16).astype(F32)))


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.00390625, 1.01171875, 1.005859375 + 2 ** -20], dtype=F32)   # exact, tie->even, tie->even, above tie
    assert list(O.f32_to_bf16_f32(x)) == [1.0, 1.0, 1.015625, 1.0078125]
