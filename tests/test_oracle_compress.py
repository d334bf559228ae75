"""Pins for the oracle's worker side (Algorithm 1: a = e + gamma*g, Delta = C_delta(a),
e' = a - Delta).  None of these needs a GPU."""
import random

import numpy as np
import pytest

from oracle import dd_ef_sgd as O
from tests import exact_arith as X


def _rand_f32(rng, n, special=True):
    v = rng.standard_normal(n).astype(np.float32) * np.float32(10.0) ** rng.integers(-6, 6, n)
    if special and n >= 8:
        v[0], v[1], v[2] = 0.0, -0.0, np.float32(1e-42)        # zeros and a subnormal
        v[3] = np.float32(-1e-42)
    return v.astype(np.float32)


def test_accumulate_is_one_fused_rounding_f32():
    rng = np.random.default_rng(1)
    n = 400
    g, e = _rand_f32(rng, n), _rand_f32(rng, n)
    # cases where rounding the product first gives a different answer than the fused op
    g[10], e[10] = np.float32(1.0 + 2 ** -12), np.float32(-1.0)
    alpha = np.float32(1.0 + 2 ** -12)
    for alpha in (np.float32(0.1), alpha, np.float32(1.0)):
        a = O.accumulate(alpha, g, e)
        for j in range(n):
            want = X.fma_f32_bits(X.f32_bits(alpha), X.f32_bits(g[j]), X.f32_bits(e[j]))
            assert int(a[j:j + 1].view(np.uint32)[0]) == want, (j, g[j], e[j])
    # the fused result differs from mul-then-add somewhere, so the test can tell them apart
    a = O.accumulate(np.float32(0.1), g, e)
    two_step = (np.float32(0.1) * g).astype(np.float32) + e
    assert np.any(a.view(np.uint32) != two_step.view(np.uint32))


def test_accumulate_bf16_widening_is_exact():
    rng = np.random.default_rng(2)
    n = 300
    gbits = rng.integers(0, 1 << 16, n).astype(np.uint16)
    gbits[(gbits & 0x7F80) == 0x7F80] = 0x3F80            # no Inf/NaN
    e = _rand_f32(rng, n)
    alpha = np.float32(0.1)
    a = O.accumulate(alpha, gbits, e)
    for j in range(n):
        want = X.fma_f32_bits(X.f32_bits(alpha), int(gbits[j]) << 16, X.f32_bits(e[j]))
        assert int(a[j:j + 1].view(np.uint32)[0]) == want


def test_magnitude_key_orders_like_abs():
    rng = np.random.default_rng(3)
    v = _rand_f32(rng, 2000)
    key = O.magnitude_key(v)
    assert key[0] == 0 and key[1] == 0                      # +0 and -0 tie
    av = np.abs(v.astype(np.float64))
    i, j = rng.integers(0, v.size, 5000), rng.integers(0, v.size, 5000)
    assert np.array_equal(key[i] < key[j], av[i] < av[j])
    assert np.array_equal(key[i] == key[j], av[i] == av[j])


def _brute_topk(vals, k):
    """Pick the largest |v| k times; equal magnitudes -> lower index (pure Python)."""
    left = list(range(len(vals)))
    out = []
    for _ in range(k):
        best = left[0]
        for j in left[1:]:
            if abs(vals[j]) > abs(vals[best]):
                best = j                                      # strict: keeps the lower index
        out.append(best)
        left.remove(best)
    return sorted(out)


@pytest.mark.parametrize("kind", ["normal", "two_valued", "all_equal", "all_zero",
                                  "signed_zero", "bf16_grid", "ramp_desc"])
def test_topk_matches_brute_force(kind):
    rng = np.random.default_rng(4)
    for d in (1, 2, 3, 31, 64, 257):
        if kind == "normal":
            v = rng.standard_normal(d)
        elif kind == "two_valued":
            v = rng.choice([0.5, -2.0], d)
        elif kind == "all_equal":
            v = np.full(d, -3.25)
        elif kind == "all_zero":
            v = np.zeros(d)
        elif kind == "signed_zero":
            v = rng.choice([0.0, -0.0, 1.0], d)
        elif kind == "bf16_grid":                           # few distinct magnitudes
            v = rng.integers(-6, 7, d) / 4.0
        else:
            v = np.arange(d, 0, -1)
        v = v.astype(np.float32)
        for k in sorted({1, max(1, d // 10), max(1, d // 2), d}):
            sel = O.topk_select(v, k)
            assert sel.tolist() == _brute_topk([float(x) for x in v], k), (kind, d, k)


def test_topk_threshold_invariants_and_contraction():
    """Selected magnitudes dominate the rest, ties split by index, and the Top-k lemma
    ||C(x) - x||^2 <= (1 - delta) ||x||^2 holds because k/d >= delta."""
    rng = np.random.default_rng(5)
    for d, delta in ((4097, 0.01), (10000, 0.1), (5000, 0.0003), (999, 1.0)):
        x = (rng.standard_t(3, d) * rng.choice([1, 1, 50], d)).astype(np.float32)
        x[rng.integers(0, d, d // 3)] = np.float32(0.75)      # a fat tie class
        k = O.k_from_delta(delta, d)
        assert k / d >= delta
        sel, vals, resid = O.compress(x, k)
        assert sel.size == k and np.all(np.diff(sel.astype(np.int64)) > 0)
        key = O.magnitude_key(x)
        mask = np.zeros(d, bool)
        mask[sel] = True
        if k < d:
            lo_in, hi_out = key[mask].min(), key[~mask].max()
            assert lo_in >= hi_out
            if lo_in == hi_out:                               # tie class cut by index
                tie = np.nonzero(key == lo_in)[0]
                assert tie[mask[tie]].max() < tie[~mask[tie]].min()
        err = float(np.sum(resid.astype(np.float64) ** 2))
        tot = float(np.sum(x.astype(np.float64) ** 2))
        assert err <= (1.0 - delta) * tot * (1 + 1e-12)


def test_error_feedback_identity_bitwise():
    """Delta and e' have disjoint supports and together are exactly a = e + gamma*g."""
    rng = np.random.default_rng(6)
    d, k = 3001, 77
    e = rng.standard_normal(d).astype(np.float32)
    g = rng.standard_normal(d).astype(np.float32)
    a = O.accumulate(np.float32(0.1), g, e)
    sel, vals, resid = O.compress(a, k)
    assert np.all(resid[sel].view(np.uint32) == 0)            # +0 where sent
    rebuilt = resid.copy()
    rebuilt[sel] = vals
    assert np.array_equal(rebuilt.view(np.uint32), a.view(np.uint32))
    assert np.array_equal(vals.view(np.uint32), a[sel].view(np.uint32))


def test_k_rule():
    # k printed with the first benchmark configuration: delta = 0.01 on d = 2^20
    assert O.k_from_delta(0.01, 1 << 20) == 10486
    assert O.k_from_delta(0.1, 100_000_000) == 10_000_000      # integer product stays
    assert O.k_from_delta(0.0001, 100_000_000) == 10_000
    assert O.k_from_delta(0.001, 124_439_808) == 124_440
    assert O.k_from_delta(0.001, 1_100_048_384) == 1_100_049
    assert O.k_from_delta(0.01, 11_689_512) == 116_896
    assert O.k_from_delta(1.0, 17) == 17
    assert O.k_from_delta(1e-9, 17) == 1
    with pytest.raises(ValueError):
        O.k_from_delta(0.0, 10)
