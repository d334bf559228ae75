"""Pins for the oracle's Random-k sparsifier: the generator against its published
known-answer vectors, the draw against brute force and against what "k entries chosen
uniformly at random" means, and the error-feedback loop built on it.  CPU only."""
import os

import numpy as np

from oracle import dd_ef_sgd as O
from oracle import random_k as R

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_philox_known_answers():
    rows = [ln.split() for ln in open(os.path.join(GOLDEN, "philox4x32_10_kat.txt"))
            if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for row in rows:
        w = [int(x, 16) for x in row]
        out = R.philox4x32_10([w[0]], [w[1]], [w[2]], [w[3]], w[4], w[5])
        assert [int(o[0]) for o in out] == w[6:10]
    # vectorised evaluation equals one-at-a-time evaluation
    c0 = np.arange(5, dtype=np.uint64)
    many = R.philox4x32_10(c0, 7, 3, 9, 11, 13)
    for q in range(5):
        one = R.philox4x32_10([q], [7], [3], [9], 11, 13)
        assert [int(m[q]) for m in many] == [int(o[0]) for o in one]


def test_priorities_follow_the_stated_counter_layout():
    d, seed, step, worker = 37, 0x1234567890ABCDEF, (5 << 32) | 17, 3
    pr = R.priorities(d, seed, step, worker)
    for j in (0, 1, 2, 3, 4, 35, 36):
        out = R.philox4x32_10([j // 4], [17], [3], [5 ^ 0x52414E44], 0x90ABCDEF, 0x12345678)
        assert int(pr[j]) == int(out[j % 4][0]) >> 9
    assert pr.max() < (1 << 23)


def test_draw_is_the_k_largest_priorities_by_brute_force():
    for d, k in ((1, 1), (5, 2), (64, 7), (257, 257), (1000, 1)):
        pr = R.priorities(d, 42, 9, 1)
        order = sorted(range(d), key=lambda j: (-int(pr[j]), j))
        assert R.randk_select(d, k, 42, 9, 1).tolist() == sorted(order[:k])


def test_draw_is_exactly_k_distinct_reproducible_and_independent():
    d, k = 100_000, 1000
    a = R.randk_select(d, k, 1, 0, 0)
    assert a.size == k and np.all(np.diff(a.astype(np.int64)) > 0) and a.max() < d
    assert np.array_equal(a, R.randk_select(d, k, 1, 0, 0))
    others = [R.randk_select(d, k, 1, 1, 0), R.randk_select(d, k, 1, 0, 1),
              R.randk_select(d, k, 2, 0, 0)]
    for b in others:                       # overlap of two independent draws is about k^2/d
        assert np.intersect1d(a, b).size < 40


def test_draw_is_uniform_over_indices():
    """Chi-square over 50 equal blocks of the index range, many draws pooled."""
    d, k, blocks = 50_000, 500, 50
    counts = np.zeros(blocks)
    for step in range(200):
        sel = R.randk_select(d, k, 7, step, 2)
        counts += np.bincount(sel // (d // blocks), minlength=blocks)
    expected = 200 * k / blocks
    chi2 = float(((counts - expected) ** 2 / expected).sum())
    assert chi2 < 90.0                      # 49 degrees of freedom: P(chi2 > 90) < 1e-3.5
    # the lowest and highest index are as likely as any other
    hits0 = sum(0 in R.randk_select(1000, 100, 3, s, 0) for s in range(300))
    hits1 = sum(999 in R.randk_select(1000, 100, 3, s, 0) for s in range(300))
    assert 10 <= hits0 <= 55 and 10 <= hits1 <= 55           # mean 30, sigma 5.2


def test_random_k_contraction_in_expectation():
    """E ||C(x) - x||^2 = (1 - k/d) ||x||^2 for a uniform draw (the compressor lemma holds with
    equality in expectation)."""
    rng = np.random.default_rng(0)
    d, k = 2000, 200
    x = rng.standard_normal(d)
    total = float((x ** 2).sum())
    kept = np.mean([float((x[R.randk_select(d, k, 5, s, 0)] ** 2).sum()) for s in range(400)])
    assert abs(kept / total - k / d) < 0.01


def test_error_feedback_with_random_k_conserves_mass_and_converges():
    rng = np.random.default_rng(1)
    T, n, d, lr, tau, delta = 10, 3, 1200, 0.1, 2, 0.05
    G = rng.standard_normal((T, n, d)).astype(np.float32)
    o = O.DDEFSGD(d, n, delta, tau, lr, compressor="randk", seed=99)
    sent = np.zeros((T, n, d))
    for t in range(T):
        out = o.step(G[t])
        for i, (sel, vals) in enumerate(out["msgs"]):
            assert np.array_equal(sel, R.randk_select(d, o.k, 99, t, i))
            sent[t, i, sel] = vals
    lhs = sent.sum(0) + o.e.astype(np.float64)
    rhs = float(np.float32(lr)) * G.astype(np.float64).sum(0)
    assert np.allclose(lhs, rhs, rtol=1e-5, atol=1e-5)
    # quadratic with identical workers: the iterates reach the minimiser
    c = np.repeat(rng.standard_normal((1, 300)).astype(np.float32), 4, axis=0)
    q = O.DDEFSGD(300, 4, 0.1, 2, 1.0 / 8, compressor="randk", seed=5)
    for _ in range(2500):
        q.step((q.x[None, :] - c).astype(np.float32))
    assert np.linalg.norm(q.x - c[0]) < 1e-3 * np.linalg.norm(c[0])
