"""The pins must be able to fail: each case plants one plausible mistake in the ORACLE (on the
CPU, never in the CUDA path) and checks that at least one pin test then raises.  A pin that
survives every mutation here would pin nothing."""
import math

import numpy as np
import pytest

from oracle import dd_ef_sgd as O
from oracle import deco_policy as P
from tests import test_oracle_algorithm as TA
from tests import test_oracle_compress as TC
from tests import test_oracle_policy as TP


def _fails(*pins):
    """True if at least one of the pin tests raises an assertion (or crashes)."""
    for pin in pins:
        try:
            pin()
        except Exception:
            return True
    return False


def _two_roundings(alpha, g, e):                       # mul then add instead of one fma
    gf = g.astype(np.float32) if g.dtype != np.uint16 else \
        (g.astype(np.uint32) << 16).view(np.float32)
    return (np.float32(alpha) * gf).astype(np.float32) + np.asarray(e, np.float32)


def _no_error_term(alpha, g, e):                       # drops e from a = e + gamma*g
    return _two_roundings(alpha, g, np.zeros_like(e))


def _topk_signed(a, k):                                # largest values instead of magnitudes
    idx = np.argsort(-a.astype(np.float64), kind="stable")[:k]
    return np.sort(idx).astype(np.uint32)


def _topk_ties_high_index(a, k):                       # equal magnitudes -> higher index
    key = O.magnitude_key(a).astype(np.int64)
    order = np.lexsort((-np.arange(a.size), -key))
    return np.sort(order[:k]).astype(np.uint32)


def _topk_smallest(a, k):
    key = O.magnitude_key(a).astype(np.int64)
    return np.sort(np.argsort(key, kind="stable")[:k]).astype(np.uint32)


def _apply_wrong_sign(x, S, scale):
    x += np.float32(scale) * S


def _aggregate_drops_last_worker(msgs, d):
    return ORIG_AGGREGATE(msgs[:-1], d)


def _aggregate_reversed_order(msgs, d):               # workers summed n-1..0
    return ORIG_AGGREGATE(msgs[::-1], d)


def _apply_two_roundings(x, S, scale):                # product rounded before the subtraction
    x -= (np.float32(scale) * S).astype(np.float32)


ORIG_AGGREGATE = O.aggregate
ORIG_STEP = O.DDEFSGD.step


COMPRESS_PINS = [TC.test_accumulate_is_one_fused_rounding_f32,
                 TC.test_accumulate_bf16_widening_is_exact,
                 lambda: TC.test_topk_matches_brute_force("normal"),
                 lambda: TC.test_topk_matches_brute_force("bf16_grid"),
                 TC.test_topk_threshold_invariants_and_contraction,
                 TC.test_error_feedback_identity_bitwise, TC.test_k_rule]
ALGO_PINS = [TA.test_delta1_tau0_is_dsgd, TA.test_delta1_is_delayed_aggregation,
             TA.test_update_t_uses_exactly_aggregate_t_minus_tau,
             TA.test_tau0_is_compression_with_error_feedback,
             TA.test_error_conservation_per_worker_and_global,
             TA.test_quadratic_converges_to_known_minimiser,
             TA.test_apply_update_is_one_fused_rounding,
             TA.test_aggregate_sums_in_worker_order_from_plus_zero]
POLICY_PINS = [TP.test_phi_degradation_conditions,
               TP.test_delta_star_is_the_largest_ratio_with_no_pipeline_bubble,
               TP.test_deco_select_matches_brute_force_and_hand_cases,
               TP.test_recurrence_matches_the_closed_forms_printed_in_the_proof,
               TP.test_t_avg_closed_form_within_the_stated_bound]


def test_pins_pass_unmutated():
    assert not _fails(*COMPRESS_PINS[:2], COMPRESS_PINS[5])


@pytest.mark.parametrize("name,target,attr,mutant,pins", [
    ("two roundings", O, "accumulate", _two_roundings, COMPRESS_PINS),
    ("error term dropped", O, "accumulate", _no_error_term, ALGO_PINS),
    ("signed top-k", O, "topk_select", _topk_signed, COMPRESS_PINS),
    ("ties to the higher index", O, "topk_select", _topk_ties_high_index, COMPRESS_PINS),
    ("smallest instead of largest", O, "topk_select", _topk_smallest, COMPRESS_PINS),
    ("k rounded down", O, "k_from_delta",
     lambda delta, d: max(1, min(int(d), int(math.floor(delta * d)))), COMPRESS_PINS),
    ("update added instead of subtracted", O, "apply_update", _apply_wrong_sign, ALGO_PINS),
    ("last worker not aggregated", O, "aggregate", _aggregate_drops_last_worker, ALGO_PINS),
    ("workers summed in reverse order", O, "aggregate", _aggregate_reversed_order,
     [TA.test_aggregate_sums_in_worker_order_from_plus_zero]),
    ("update with two roundings", O, "apply_update", _apply_two_roundings,
     [TA.test_apply_update_is_one_fused_rounding]),
    ("phi without the staleness power", P, "phi",
     lambda delta, tau: (1 - delta) / delta, POLICY_PINS),
    ("phi with (1 - delta)^tau", P, "phi",
     lambda delta, tau: (1 - delta) / (delta * (1 - delta) ** tau), POLICY_PINS),
    ("delta* without the compute cap", P, "delta_star",
     lambda tau, V, a, b, Tc: min(max(0.0, (tau * Tc - b) * a / V), 1.0), POLICY_PINS),
    ("delta* with latency added", P, "delta_star",
     lambda tau, V, a, b, Tc: min(max(0.0, (tau * Tc + b) * a / V), Tc * a / V, 1.0), POLICY_PINS),
    ("T_avg without the latency term", P, "t_avg",
     lambda delta, tau, V, a, b, Tc: max((Tc + delta * V / a) / (tau + 1), delta * V / a, Tc),
     POLICY_PINS),
    ("T_avg divided by tau", P, "t_avg",
     lambda delta, tau, V, a, b, Tc: max((Tc + b + delta * V / a) / max(tau, 1), delta * V / a, Tc),
     POLICY_PINS),
])
def test_planted_mistake_is_caught(monkeypatch, name, target, attr, mutant, pins):
    monkeypatch.setattr(target, attr, mutant)
    assert _fails(*pins), "no pin noticed: " + name


def test_staleness_off_by_one_is_caught(monkeypatch):
    def early(self, g):                                   # applies S_{t-tau+1}
        real_tau = self.tau
        self.tau = max(0, real_tau - 1)
        try:
            return ORIG_STEP(self, g)
        finally:
            self.tau = real_tau
    monkeypatch.setattr(O.DDEFSGD, "step", early)
    assert _fails(TA.test_delta1_is_delayed_aggregation,
                  TA.test_update_t_uses_exactly_aggregate_t_minus_tau)


def test_recurrence_mistakes_are_caught(monkeypatch):
    def no_latency(delta, tau, V, a, b, Tc, E):           # TC_k = TM_k
        return P_ORIG(delta, tau, V, a, 0.0, Tc, E)
    P_ORIG = P.pipeline_times
    monkeypatch.setattr(P, "pipeline_times", no_latency)
    assert _fails(TP.test_recurrence_matches_the_closed_forms_printed_in_the_proof,
                  TP.test_t_avg_closed_form_within_the_stated_bound)
