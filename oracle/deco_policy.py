"""DeCo (Algorithm 3), phi, delta*(tau) and the iteration-time model (Theorem 3) on the CPU.

TEST INFRASTRUCTURE ONLY.  Float64 throughout, written in the paper's notation:
V_g gradient volume (bits), a_bar average bandwidth (bits/s), b end-to-end latency (s),
T_comp computation time per iteration (s), tau staleness, delta compression ratio.

Readings where Algorithm 3 and the text leave a gap:
  * the remark on delta*(tau) clamps at 0 while Algorithm 3 does not; a candidate with
    delta <= 0 has phi = +inf and is skipped;
  * the set is walked from the largest tau down with "phi <= phi_min", so equal phi goes to
    the smaller tau, as the text asks ("choose the smallest tau");
  * if no tau of the range is feasible, tau = ceil(b/T_comp) + 1 with its delta*(tau);
  * non_iid swaps phi for phi' = phi / delta (remark on phi).
"""
import math


def phi(delta, tau):
    """Convergence factor phi = (1 - delta) / (delta * (1 - delta/2)^tau) of Theorem 1."""
    return (1.0 - delta) / (delta * (1.0 - delta / 2.0) ** tau)


def phi_prime(delta, tau):
    """phi' = (1 - delta) / (delta^2 * (1 - delta/2)^tau), the non-IID factor."""
    return (1.0 - delta) / (delta * delta * (1.0 - delta / 2.0) ** tau)


def delta_star(tau, V_g, a_bar, b, T_comp):
    """Locally optimal ratio for a given tau (remark after Theorem 3)."""
    return min(max(0.0, (tau * T_comp - b) * a_bar / V_g), T_comp * a_bar / V_g, 1.0)


def tau_range(V_g, a_bar, b, T_comp):
    lo = math.ceil(b / T_comp)
    hi = math.ceil((b + V_g / a_bar) / T_comp)
    return lo, hi


def deco_select(V_g, a_bar, b, T_comp, non_iid=False):
    """Algorithm 3: (tau*, delta*) minimising phi over the tau range, ties to the smaller tau."""
    lo, hi = tau_range(V_g, a_bar, b, T_comp)
    f = phi_prime if non_iid else phi
    best = None
    phi_min = math.inf
    for tau in range(hi, lo - 1, -1):
        delta = delta_star(tau, V_g, a_bar, b, T_comp)
        if delta <= 0.0:
            continue
        val = f(delta, tau)
        if val <= phi_min:
            phi_min = val
            best = (tau, delta)
    if best is None:
        tau = lo + 1
        best = (tau, delta_star(tau, V_g, a_bar, b, T_comp))
    return best


def t_avg(delta, tau, V_g, a_bar, b, T_comp):
    """Theorem 3: estimated average time per iteration."""
    t_delta = delta * V_g / a_bar
    return max((T_comp + b + t_delta) / (tau + 1), t_delta, T_comp)


def pipeline_times(delta, tau, V_g, a_bar, b, T_comp, E):
    """The recurrence in the proof of Theorem 3 run for E iterations.

        TC_k     = TM_k + b
        TS_{k+1} = T_comp  + max(TC_{k-tau}, TS_k)
        TM_{k+1} = delta*V_g/a_bar + max(TM_k, TS_{k+1})
    with TS_0 = TM_0 = 0 and TC_k = 0 for k <= 0.  Returns (TS, TM, TC) lists of length E+1."""
    t_delta = delta * V_g / a_bar
    TS = [0.0] * (E + 1)
    TM = [0.0] * (E + 1)
    TC = [0.0] * (E + 1)

    def tc(k):
        return TC[k] if k > 0 else 0.0

    for k in range(E):
        TS[k + 1] = T_comp + max(tc(k - tau), TS[k])
        TM[k + 1] = t_delta + max(TM[k], TS[k + 1])
        TC[k + 1] = TM[k + 1] + b
    return TS, TM, TC


def build_lut(V_g, a_min, a_max, b, T_comp, points=20, non_iid=False):
    """Look-up table of the implementation section: `points` linearly spaced bandwidths in
    [a_min, a_max], each with its DeCo decision for the measured b."""
    if points < 2:
        grid = [a_min]
    else:
        grid = [a_min + (a_max - a_min) * i / (points - 1) for i in range(points)]
    return [(a, ) + deco_select(V_g, a, b, T_comp, non_iid) for a in grid]


def lut_lookup(lut, a_bar, V_g, b, T_comp, non_iid=False):
    """Nearest sample point inside the profiled range, online DeCo outside it."""
    if a_bar < lut[0][0] or a_bar > lut[-1][0]:
        return deco_select(V_g, a_bar, b, T_comp, non_iid)
    best = min(lut, key=lambda row: (abs(row[0] - a_bar), row[0]))
    return best[1], best[2]
