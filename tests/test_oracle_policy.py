"""Pins for the oracle's DeCo policy (Algorithm 3), phi, delta*(tau) and the iteration-time
model (Theorem 3 and the recurrence of its proof).  CPU only."""
import math
import os
import random

import pytest

from oracle import deco_policy as P

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_phi_degradation_conditions():
    """delta = 1 gives phi = 0; tau = 0 gives phi = (1 - delta)/delta (degradation remark)."""
    for tau in (0, 1, 5, 40):
        assert P.phi(1.0, tau) == 0.0
    for delta in (0.5, 0.1, 0.003):
        assert P.phi(delta, 0) == pytest.approx((1 - delta) / delta, rel=1e-15)
    # one value by hand: delta = 0.5, tau = 2 -> 0.5 / (0.5 * 0.75^2) = 16/9
    assert P.phi(0.5, 2) == pytest.approx(16.0 / 9.0, rel=1e-15)
    assert P.phi_prime(0.5, 2) == pytest.approx(32.0 / 9.0, rel=1e-15)
    # phi grows with tau and shrinks with delta
    assert P.phi(0.1, 3) > P.phi(0.1, 2) and P.phi(0.2, 3) < P.phi(0.1, 3)


def test_delta_star_is_the_largest_ratio_with_no_pipeline_bubble():
    """T_avg(tau, delta*(tau)) = T_comp, and any larger delta is slower (remark on delta*)."""
    rnd = random.Random(20)
    for _ in range(2000):
        Tc = rnd.uniform(0.01, 1.0)
        b = rnd.uniform(0.0, 1.0)
        a = 10 ** rnd.uniform(8, 10)
        Vg = 32 * 10 ** rnd.uniform(6, 9)
        tau = rnd.randint(0, 30)
        ds = P.delta_star(tau, Vg, a, b, Tc)
        assert 0.0 <= ds <= 1.0
        if ds <= 0.0:
            assert tau * Tc <= b
            continue
        assert P.t_avg(ds, tau, Vg, a, b, Tc) == pytest.approx(Tc, rel=1e-12)
        if ds < 1.0:
            assert P.t_avg(min(1.0, ds * 1.05), tau, Vg, a, b, Tc) > Tc * (1 + 1e-9)


def _brute_deco(Vg, a, b, Tc):
    """Ascending walk with strict '<': first minimiser = smallest tau."""
    lo = math.ceil(b / Tc)
    hi = math.ceil((b + Vg / a) / Tc)
    best, best_phi = None, math.inf
    for tau in range(lo, hi + 1):
        delta = min((tau * Tc - b) * a / Vg, Tc * a / Vg, 1.0)
        if delta <= 0:
            continue
        ph = (1 - delta) / (delta * (1 - delta / 2) ** tau)
        if ph < best_phi:
            best, best_phi = (tau, delta), ph
    return best


def test_deco_select_matches_brute_force_and_hand_cases():
    rnd = random.Random(21)
    for _ in range(3000):
        Tc = rnd.uniform(0.01, 0.5)
        b = rnd.uniform(0.0, 0.5)
        a = 10 ** rnd.uniform(7.5, 10.5)
        Vg = 32 * 10 ** rnd.uniform(6, 9)
        got = P.deco_select(Vg, a, b, Tc)
        want = _brute_deco(Vg, a, b, Tc)
        if want is not None:
            assert got[0] == want[0] and got[1] == pytest.approx(want[1], rel=1e-12)
    with open(os.path.join(GOLDEN, "deco_hand_cases.txt")) as fh:
        rows = [ln.split() for ln in fh if ln.strip() and not ln.startswith("#")]
    assert len(rows) == 3
    for a, b, tau, delta in rows:
        got = P.deco_select(3.2e9, float(a), float(b), 0.05)
        assert got[0] == int(tau) and got[1] == pytest.approx(float(delta), rel=1e-12)


def test_deco_select_edge_cases():
    # latency a multiple of T_comp: the first candidate has delta = 0 and is skipped
    tau, delta = P.deco_select(3.2e9, 1e9, 0.10, 0.05)
    assert tau == 3 and delta > 0
    # bandwidth so high that the whole gradient fits: delta = 1, phi = 0 wins
    tau, delta = P.deco_select(3.2e6, 1e10, 0.01, 0.05)
    assert delta == 1.0 and tau == 1
    # non-IID factor never picks a smaller delta than the IID one at equal tau range
    t1, d1 = P.deco_select(3.2e9, 5e9, 0.03, 0.05, non_iid=False)
    t2, d2 = P.deco_select(3.2e9, 5e9, 0.03, 0.05, non_iid=True)
    assert d2 >= d1


def test_recurrence_matches_the_closed_forms_printed_in_the_proof():
    """Proof of Theorem 3: explicit TS_i / TM_i per regime."""
    Vg, a = 1e9, 1e9                                   # t_delta = delta seconds
    # Case 1: T_comp > t_delta and tau*T_comp > t_delta + b  ->  TS_k = k*T_comp
    Tc, b, td, tau, E = 0.5, 0.3, 0.2, 2, 40
    TS, TM, TC = P.pipeline_times(td, tau, Vg, a, b, Tc, E)
    for k in range(1, E + 1):
        assert TS[k] == pytest.approx(k * Tc, rel=1e-12)
        assert TM[k] == pytest.approx(td + k * Tc, rel=1e-12)
    assert TC[E] == pytest.approx(td + E * Tc + b, rel=1e-12)
    # Case 3: T_comp > t_delta and tau*T_comp <= t_delta + b
    Tc, b, td, tau = 0.5, 1.4, 0.2, 3
    TS, TM, TC = P.pipeline_times(td, tau, Vg, a, b, Tc, 4 * tau + 4)
    for i in range(1, tau + 2):
        assert TS[i] == pytest.approx(i * Tc) and TM[i] == pytest.approx(td + i * Tc)
    for i in range(tau + 2, 2 * tau + 3):
        assert TS[i] == pytest.approx(td + b + (i - tau) * Tc)
        assert TM[i] == pytest.approx(2 * td + b + (i - tau) * Tc)
    period = Tc + b + td                                # (tau+1)-periodic increments
    for i in range(1, 2 * tau + 3):
        assert TS[i + tau + 1] - TS[i] == pytest.approx(period)
    # Case 4: T_comp < t_delta and tau*t_delta <= T_comp + b
    Tc, b, td, tau = 0.2, 1.5, 0.5, 3
    TS, TM, TC = P.pipeline_times(td, tau, Vg, a, b, Tc, 4 * tau + 4)
    for i in range(1, tau + 2):
        assert TS[i] == pytest.approx(i * Tc) and TM[i] == pytest.approx(i * td + Tc)
    for i in range(tau + 2, 2 * tau + 3):
        assert TM[i] == pytest.approx((b + Tc + td) + Tc + (i - tau - 1) * td)
    # Case 2: t_delta > T_comp and tau*t_delta > T_comp + b -> TM_i = T_comp + i*t_delta
    Tc, b, td, tau = 0.2, 0.3, 0.5, 2
    TS, TM, TC = P.pipeline_times(td, tau, Vg, a, b, Tc, 30)
    for i in range(1, 31):
        assert TM[i] == pytest.approx(Tc + i * td)


def test_t_avg_closed_form_within_the_stated_bound():
    """|TC_E - E*T_avg| <= b + min(T_comp, t_delta) for every regime (summary of the proof)."""
    rnd = random.Random(22)
    for _ in range(3000):
        Tc = rnd.uniform(0.01, 1.0)
        b = rnd.uniform(0.0, 2.0)
        td = rnd.uniform(0.001, 2.0)
        tau = rnd.randint(0, 12)
        E = rnd.randint(max(10, 3 * tau + 3), 300)
        TS, TM, TC = P.pipeline_times(td, tau, 1e9, 1e9, b, Tc, E)
        est = P.t_avg(td, tau, 1e9, 1e9, b, Tc)
        assert abs(TC[E] - E * est) <= (b + min(Tc, td)) * (1 + 1e-9) + 1e-12


def test_lut_nearest_and_fallback():
    Vg, b, Tc = 3.2e9, 0.1, 0.05
    lut = P.build_lut(Vg, 0.5e9, 2.0e9, b, Tc, points=20)
    assert len(lut) == 20 and lut[0][0] == 0.5e9 and lut[-1][0] == pytest.approx(2.0e9)
    step = (2.0e9 - 0.5e9) / 19
    a = 0.5e9 + 3.4 * step                                   # nearest sample is #3
    assert P.lut_lookup(lut, a, Vg, b, Tc) == (lut[3][1], lut[3][2])
    out = P.lut_lookup(lut, 5e9, Vg, b, Tc)                  # outside: online decision
    assert out == P.deco_select(Vg, 5e9, b, Tc)
