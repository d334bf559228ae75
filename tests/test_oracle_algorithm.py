"""Pins for the whole DD-EF-SGD loop of the oracle (Algorithm 1) against what the paper and
the mathematics fix: the degradation conditions, the staleness boundary, error conservation
(the virtual-sequence identities) and convergence on a quadratic.  CPU only."""
import numpy as np

from oracle import dd_ef_sgd as O


def _grads(rng, steps, n, d):
    return rng.standard_normal((steps, n, d)).astype(np.float32)


def test_delta1_tau0_is_dsgd():
    """Degradation conditions (delta = 1 and tau = 0): x_{t+1} = x_t - (gamma/n) sum_i g_t^i."""
    rng = np.random.default_rng(10)
    T, n, d, lr = 7, 4, 500, 0.05
    G = _grads(rng, T, n, d)
    x0 = rng.standard_normal(d).astype(np.float32)
    o = O.DDEFSGD(d, n, 1.0, 0, lr, x0=x0)
    ref = x0.astype(np.float64)
    for t in range(T):
        o.step(G[t])
        ref = ref - (float(np.float32(lr)) / n) * G[t].astype(np.float64).sum(0)
        assert np.allclose(o.x, ref, rtol=1e-6, atol=1e-6)
        assert np.all(o.e == 0)                                  # nothing is left behind
    assert np.allclose(o.x64, ref, rtol=1e-7, atol=1e-7)


def test_delta1_is_delayed_aggregation():
    """delta = 1: x_{t+1} = x_t - (gamma/n) sum_i g_{t-tau}^i, nothing applied while t < tau."""
    rng = np.random.default_rng(11)
    T, n, d, lr, tau = 9, 3, 300, 0.1, 3
    G = _grads(rng, T, n, d)
    o = O.DDEFSGD(d, n, 1.0, tau, lr)
    ref = np.zeros(d)
    for t in range(T):
        out = o.step(G[t])
        if t - tau >= 0:
            ref = ref - (float(np.float32(lr)) / n) * G[t - tau].astype(np.float64).sum(0)
            assert out["applied"] == [t - tau]
        else:
            assert out["applied"] == [] and np.all(o.x == 0)
        assert np.allclose(o.x, ref, rtol=1e-6, atol=1e-6)
    assert [s for s, _ in o.in_flight()] == list(range(T - tau, T))


def test_update_t_uses_exactly_aggregate_t_minus_tau():
    """Step-tagged gradients g_t = (t+1)*c reveal which step each update came from."""
    n, d, tau, lr = 2, 64, 2, 0.5
    c = np.linspace(1.0, 2.0, d).astype(np.float32)
    o = O.DDEFSGD(d, n, 1.0, tau, lr)
    prev = o.x.copy()
    for t in range(8):
        g = np.stack([(t + 1) * c] * n).astype(np.float32)
        o.step(g)
        moved = (prev - o.x).astype(np.float64)
        if t < tau:
            assert np.all(moved == 0)
        else:
            tag = moved / (lr * c)                               # = (t - tau + 1)
            assert np.allclose(tag, t - tau + 1, rtol=1e-5)
        prev = o.x.copy()


def test_tau0_is_compression_with_error_feedback():
    """tau = 0: x_{t+1} = x_t - (1/n) sum_i Delta_t^i with Delta = C_delta(e + gamma g)."""
    rng = np.random.default_rng(12)
    T, n, d, lr = 6, 4, 2000, 0.1
    G = _grads(rng, T, n, d)
    o = O.DDEFSGD(d, n, 0.05, 0, lr)
    sent = np.zeros(d)
    for t in range(T):
        out = o.step(G[t])
        assert out["applied"] == [t]
        for sel, vals in out["msgs"]:
            assert sel.size == O.k_from_delta(0.05, d)
            sent[sel] += vals.astype(np.float64)
        assert np.allclose(o.x, -sent / n, rtol=1e-5, atol=1e-6)


def test_error_conservation_per_worker_and_global():
    """Per worker: sum_s Delta_s^i + e_T^i = gamma sum_s g_s^i (telescoped error feedback).
    Globally: x_0 - x_T = (1/n) * (messages of steps 0 .. T-tau-1), the rest is in flight."""
    rng = np.random.default_rng(13)
    T, n, d, lr, tau, delta = 12, 3, 1500, 0.1, 3, 0.02
    G = _grads(rng, T, n, d)
    o = O.DDEFSGD(d, n, delta, tau, lr)
    sent = np.zeros((T, n, d))
    for t in range(T):
        out = o.step(G[t])
        for i, (sel, vals) in enumerate(out["msgs"]):
            sent[t, i, sel] = vals
    lhs = sent.sum(0) + o.e.astype(np.float64)
    rhs = float(np.float32(lr)) * G.astype(np.float64).sum(0)
    assert np.allclose(lhs, rhs, rtol=1e-5, atol=1e-5)
    applied = sent[:T - tau].sum((0, 1)) / n
    assert np.allclose(-o.x.astype(np.float64), applied, rtol=1e-5, atol=1e-6)
    scale32 = float(np.float32(1.0) / np.float32(n))             # the shadow uses the fp32 scale
    assert np.allclose(-o.x64, applied * n * scale32, rtol=1e-9, atol=1e-9)
    flight = sum(S.astype(np.float64) for _, S in o.in_flight())
    assert np.allclose(flight, sent[T - tau:].sum((0, 1)), rtol=1e-5, atol=1e-6)


def test_tau_change_drains_cache_exactly_once():
    rng = np.random.default_rng(14)
    n, d = 2, 200
    o = O.DDEFSGD(d, n, 0.1, 3, 0.1)
    seen = []
    plan = {4: (0.1, 1), 7: (0.2, 4), 12: (0.05, 0)}
    for t in range(16):
        if t in plan:
            o.set_policy(*plan[t])
        out = o.step(rng.standard_normal((n, d)).astype(np.float32))
        assert all(s <= t - o.tau for s in out["applied"])
        assert out["k"] == O.k_from_delta(o.delta, d)
        seen += out["applied"]
    assert seen == sorted(set(seen))                              # once each, oldest first
    assert seen + [s for s, _ in o.in_flight()] == list(range(16))


def test_stepsize_inside_or_outside_compressor_agree():
    """C_delta is positively homogeneous, so for a constant stepsize moving gamma from the
    worker to the server changes only rounding (tie-free inputs)."""
    rng = np.random.default_rng(15)
    T, n, d, lr = 8, 3, 1000, 0.25          # power-of-two stepsize: scaling is exact
    G = _grads(rng, T, n, d)
    a = O.DDEFSGD(d, n, 0.05, 2, lr, lr_in_compress=True)
    b = O.DDEFSGD(d, n, 0.05, 2, lr, lr_in_compress=False)
    for t in range(T):
        ra, rb = a.step(G[t]), b.step(G[t])
        for (sa, va), (sb, vb) in zip(ra["msgs"], rb["msgs"]):
            assert np.array_equal(sa, sb)
            assert np.array_equal(va, np.float32(lr) * vb)
    assert np.allclose(a.x, b.x, rtol=1e-6, atol=1e-7)


def test_quadratic_converges_to_known_minimiser():
    """f_i(x) = 0.5 ||x - c_i||^2 (L = 1, minimiser mean(c_i)) with gamma <= 1/(4 L tau).
    Identical workers (zeta = 0, sigma = 0): the iterates reach the minimiser.  Heterogeneous
    workers: a constant stepsize leaves a neighbourhood that shrinks with gamma (the zeta
    terms of Theorem 1 carry a factor gamma)."""
    rng = np.random.default_rng(16)
    n, d, tau, delta = 4, 400, 2, 0.1

    def run(c, lr, steps):
        o = O.DDEFSGD(d, n, delta, tau, lr)
        for _ in range(steps):
            o.step((o.x[None, :] - c).astype(np.float32))         # exact local gradients
        x_star = c.astype(np.float64).mean(0)
        return np.linalg.norm(o.x - x_star) / np.linalg.norm(x_star)

    same = np.repeat(rng.standard_normal((1, d)).astype(np.float32), n, axis=0)
    assert run(same, 1.0 / (4 * tau), 1500) < 1e-4
    mixed = rng.standard_normal((n, d)).astype(np.float32)
    coarse, fine = run(mixed, 1.0 / (4 * tau), 800), run(mixed, 1.0 / (16 * tau), 3000)
    assert fine < 0.5 * coarse


def test_apply_update_is_one_fused_rounding():
    """Server update of Algorithm 1, x <- x - scale*S, pinned bit for bit against exact
    rational arithmetic with a single rounding (no fmaf is called on the checking side).  The
    triples include ones where rounding the product scale*S first gives different bits."""
    from tests import exact_arith as X
    rng = np.random.default_rng(7)
    m = 300
    S = (rng.standard_normal(m) * 10.0 ** rng.integers(-5, 5, m)).astype(np.float32)
    x = (rng.standard_normal(m) * 10.0 ** rng.integers(-5, 5, m)).astype(np.float32)
    # crafted: scale*S needs more than 24 bits and nearly cancels x
    S[0], x[0] = np.float32(1.0 + 2 ** -12), np.float32(1.0 / 3.0)
    S[1], x[1] = np.float32(3.0 + 2 ** -20), np.float32(1.0)
    S[2], x[2] = np.float32(0.0), np.float32(-0.0)
    S[3], x[3] = np.float32(1e-42), np.float32(-1e-43)           # subnormals
    differs = 0
    for scale in (np.float32(1.0) / np.float32(3.0), np.float32(0.1) / np.float32(4.0),
                  np.float32(0.25), np.float32(1.0 + 2 ** -12)):
        got = x.copy()
        O.apply_update(got, S.copy(), scale)
        neg = X.f32_bits(float(-np.float32(scale)))
        for j in range(m):
            want = X.fma_f32_bits(neg, X.f32_bits(float(S[j])), X.f32_bits(float(x[j])))
            assert int(got[j:j + 1].view(np.uint32)[0]) == want, (float(scale), j, S[j], x[j])
        two_step = x - (np.float32(scale) * S).astype(np.float32)
        differs += int(np.sum(got.view(np.uint32) != two_step.view(np.uint32)))
    assert differs > 0          # the pin can tell one rounding from two


def _sequential_f32_sum_bits(terms):
    """Bits of ((0 + t0) + t1) + ... with one rounding per addition, by exact arithmetic."""
    from tests import exact_arith as X
    one = X.f32_bits(1.0)
    acc = 0                                                  # +0
    for t in terms:
        acc = X.fma_f32_bits(one, X.f32_bits(float(t)), acc)   # 1*t + acc, rounded once
    return acc


def test_aggregate_sums_in_worker_order_from_plus_zero():
    """S = sum_i Delta^i is taken in fp32 in worker order 0..n-1 starting from +0 (fp32 addition
    is not associative, so the order is part of the result).  Three workers send the same index
    with values whose sum depends on the order; the expected bits come from exact arithmetic
    with one rounding per addition in the order 0, 1, 2, and differ from the reversed order."""
    d = 6
    big, small = np.float32(2.0 ** 24), np.float32(1.0)
    cases = [
        (np.array([big, small, small], np.float32)),           # (2^24 + 1) + 1 = 2^24 ; reversed: 2^24 + 2
        (np.array([small, small, big], np.float32)),
        (np.array([np.float32(1e8), np.float32(-1e8), np.float32(3.25)], np.float32)),
        (np.array([np.float32(0.1), np.float32(0.2), np.float32(-0.3)], np.float32)),
    ]
    order_matters = 0
    for vals in cases:
        msgs = [(np.array([4], np.uint32), vals[i:i + 1].copy()) for i in range(3)]
        # a second index sent only by worker 1: must come out as 0 + v, i.e. v itself
        msgs[1] = (np.array([2, 4], np.uint32), np.array([np.float32(-0.0), vals[1]], np.float32))
        S, S64 = O.aggregate(msgs, d)
        assert int(S[4:5].view(np.uint32)[0]) == _sequential_f32_sum_bits(vals)
        assert int(S[2:3].view(np.uint32)[0]) == 0              # +0 + -0 = +0
        assert S64[4] == float(vals[0]) + float(vals[1]) + float(vals[2])     # float64 shadow
        assert np.all(S[[0, 1, 3, 5]].view(np.uint32) == 0)
        order_matters += _sequential_f32_sum_bits(vals) != _sequential_f32_sum_bits(vals[::-1])
    assert order_matters >= 2   # the pin can tell the order 0..n-1 from its reverse
