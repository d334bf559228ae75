"""Pins of the oracle's per-layer Top-k variant (CPU only): brute force per range, reduction to
the global rule for a single layer, the per-layer counts, and the conservation invariant."""
import numpy as np

from oracle import dd_ef_sgd as O


def _brute_layer(a, lo, hi, k):
    """k largest |a[lo:hi]| by an explicit stable ordering: magnitude descending, index ascending."""
    order = sorted(range(lo, hi), key=lambda j: (-abs(float(a[j])), j))
    return sorted(order[:k])


def test_per_layer_selection_is_the_brute_force_choice_in_every_range():
    rng = np.random.default_rng(5)
    offsets = [0, 7, 8, 40, 41, 300, 1000]
    for delta in (0.01, 0.1, 0.34, 1.0):
        a = rng.standard_normal(1000).astype(np.float32)
        a[8:40] *= 100.0                                   # one loud layer
        a[300:400] = np.float32(0.5)                       # ties inside a layer
        sel = O.topk_select_per_layer(a, offsets, delta)
        want = []
        for lo, hi in zip(offsets[:-1], offsets[1:]):
            want += _brute_layer(a, lo, hi, O.k_from_delta(delta, hi - lo))
        assert sel.tolist() == want
        # the loud layer would swallow a global Top-k of the same size
        glob = O.topk_select(a, len(want))
        if delta < 0.3:
            assert set(glob.tolist()) != set(want)


def test_single_layer_reduces_to_the_global_rule():
    rng = np.random.default_rng(6)
    g = rng.standard_normal((4, 3, 500)).astype(np.float32)
    a = O.DDEFSGD(500, 3, 0.05, 2, 0.1)
    b = O.DDEFSGD(500, 3, 0.05, 2, 0.1, layer_offsets=[0, 500])
    for t in range(4):
        ra, rb = a.step(g[t]), b.step(g[t])
        for (sa, va), (sb, vb) in zip(ra["msgs"], rb["msgs"]):
            assert np.array_equal(sa, sb) and np.array_equal(va, vb)
    assert np.array_equal(a.x, b.x) and np.array_equal(a.e, b.e)


def test_counts_per_layer_and_conservation():
    """Every message holds exactly k(delta, d_l) entries of each layer, and what the workers
    produced is either applied, cached at the server or still in the residuals:
    x0 - x_T = (1/n) * sum(applied), and n*(x0 - x_T) + sum(in flight) + sum_i e_i =
    gamma * sum_t sum_i g_t^i, up to fp32 rounding."""
    rng = np.random.default_rng(7)
    offsets, n, d, lr, tau = [0, 64, 1064, 1100, 4000], 3, 4000, 0.1, 2
    o = O.DDEFSGD(d, n, 0.02, tau, lr, layer_offsets=offsets)
    total = np.zeros(d)
    for t in range(9):
        if t == 5:
            o.set_policy(0.1, 1)
        g = rng.standard_normal((n, d)).astype(np.float32)
        total += float(np.float32(lr)) * g.astype(np.float64).sum(axis=0)
        r = o.step(g)
        for sel, _ in r["msgs"]:
            assert sel.size == o.k
            for lo, hi in zip(offsets[:-1], offsets[1:]):
                inside = np.count_nonzero((sel >= lo) & (sel < hi))
                assert inside == O.k_from_delta(o.delta, hi - lo)
    flight = sum(S.astype(np.float64) for _, S in o.in_flight())
    lhs = -n * o.x64 + flight + o.e.astype(np.float64).sum(axis=0)
    assert np.allclose(lhs, total, rtol=0, atol=1e-4)
