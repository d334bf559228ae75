// Host-side policy: DeCo (Algorithm 3), the locally optimal ratio delta*(tau), the
// convergence factor phi and the iteration-time estimate of Theorem 3.  Double precision,
// no device code.
#include <cmath>
#include <limits>

#include "deco.h"

namespace {

double phi_of(double delta, uint32_t tau, bool non_iid)
{
    // phi = (1 - delta) / (delta * (1 - delta/2)^tau);  phi' = phi / delta
    double v = (1.0 - delta) / (delta * std::pow(1.0 - 0.5 * delta, static_cast<double>(tau)));
    return non_iid ? v / delta : v;
}

double delta_star_of(double tau, double Vg, double a, double b, double Tc)
{
    double by_latency = (tau * Tc - b) * a / Vg;    // transmission hidden behind tau iterations
    double by_compute = Tc * a / Vg;                // transmission no longer than one iteration
    double v = by_latency < by_compute ? by_latency : by_compute;
    if (v > 1.0) v = 1.0;
    if (v < 0.0) v = 0.0;
    return v;
}

}  // namespace

extern "C" deco_status deco_policy_select(double Vg, double a, double b, double Tc,
                                          uint32_t tau_cap, int32_t non_iid, uint32_t *tau_out,
                                          double *delta_out)
{
    if (!tau_out || !delta_out) return DECO_ERR_INVALID_ARG;
    if (!(Vg > 0.0) || !(a > 0.0) || !(b >= 0.0) || !(Tc > 0.0)) return DECO_ERR_INVALID_ARG;
    if (!std::isfinite(Vg) || !std::isfinite(a) || !std::isfinite(b) || !std::isfinite(Tc))
        return DECO_ERR_INVALID_ARG;
    const double lo_f = std::ceil(b / Tc), hi_f = std::ceil((b + Vg / a) / Tc);
    if (hi_f > 4.0e9) return DECO_ERR_INVALID_ARG;
    const uint64_t lo = static_cast<uint64_t>(lo_f), hi = static_cast<uint64_t>(hi_f);
    double phi_min = std::numeric_limits<double>::infinity();
    bool found = false;
    uint64_t best_tau = 0;
    double best_delta = 0.0;
    // Above the tau where the latency term stops binding, delta stays at its cap and phi only
    // grows with tau, so the walk may start there instead of at `hi`: same decision, O(1).
    uint64_t start = hi;
    {
        const double cap = std::fmin(Tc * a / Vg, 1.0);
        const double t_flat = std::ceil((cap * Vg / a + b) / Tc) + 1.0;   // delta*(t) == cap for t >= t_flat
        if (t_flat >= lo_f && t_flat < hi_f) start = static_cast<uint64_t>(t_flat);
    }
    for (uint64_t tau = start + 1; tau-- > lo;) {
        const double delta = delta_star_of(static_cast<double>(tau), Vg, a, b, Tc);
        if (delta <= 0.0) continue;
        const double ph = phi_of(delta, static_cast<uint32_t>(tau), non_iid != 0);
        if (ph <= phi_min) {
            phi_min = ph;
            best_tau = tau;
            best_delta = delta;
            found = true;
        }
    }
    if (!found) {
        best_tau = lo + 1;
        best_delta = delta_star_of(static_cast<double>(best_tau), Vg, a, b, Tc);
    }
    if (tau_cap != 0 && best_tau > tau_cap) {
        best_tau = tau_cap;
        best_delta = delta_star_of(static_cast<double>(best_tau), Vg, a, b, Tc);
    }
    *tau_out = static_cast<uint32_t>(best_tau);
    *delta_out = best_delta;
    return DECO_OK;
}

extern "C" double deco_t_avg(double delta, uint32_t tau, double Vg, double a, double b, double Tc)
{
    if (!(delta >= 0.0) || !(Vg > 0.0) || !(a > 0.0) || !(b >= 0.0) || !(Tc > 0.0)) return -1.0;
    const double t_delta = delta * Vg / a;
    double v = (Tc + b + t_delta) / (static_cast<double>(tau) + 1.0);
    if (t_delta > v) v = t_delta;
    if (Tc > v) v = Tc;
    return v;
}

extern "C" uint64_t deco_k_from_delta(double delta, uint64_t d)
{
    if (!(delta > 0.0) || !(delta <= 1.0) || d == 0) return 0;
    const double prod = delta * static_cast<double>(d);
    const double nearest = std::nearbyint(prod);
    double kf = (std::fabs(prod - nearest) <= 1e-6) ? nearest : std::ceil(prod);
    if (kf < 1.0) kf = 1.0;
    uint64_t k = static_cast<uint64_t>(kf);
    if (k > d) k = d;
    return k;
}

extern "C" deco_status deco_lut_build(double Vg, double a_min, double a_max, double b, double Tc,
                                      uint32_t points, uint32_t tau_cap, int32_t non_iid,
                                      deco_lut_entry *lut)
{
    if (!lut || points == 0 || !(a_min > 0.0) || !(a_max >= a_min)) return DECO_ERR_INVALID_ARG;
    for (uint32_t q = 0; q < points; ++q) {
        const double a = points < 2 ? a_min
                                    : a_min + (a_max - a_min) * static_cast<double>(q) /
                                                  static_cast<double>(points - 1);
        uint32_t tau = 0;
        double delta = 0.0;
        const deco_status st = deco_policy_select(Vg, a, b, Tc, tau_cap, non_iid, &tau, &delta);
        if (st != DECO_OK) return st;
        lut[q].a_bps = a;
        lut[q].delta = delta;
        lut[q].tau = tau;
        lut[q].reserved = 0;
    }
    return DECO_OK;
}

extern "C" deco_status deco_lut_lookup(const deco_lut_entry *lut, uint32_t points, double a_bar,
                                       double Vg, double b, double Tc, uint32_t tau_cap,
                                       int32_t non_iid, uint32_t *tau_out, double *delta_out)
{
    if (!lut || points == 0 || !tau_out || !delta_out || !(a_bar > 0.0)) return DECO_ERR_INVALID_ARG;
    if (a_bar < lut[0].a_bps || a_bar > lut[points - 1].a_bps)     // outside the profiled range
        return deco_policy_select(Vg, a_bar, b, Tc, tau_cap, non_iid, tau_out, delta_out);
    uint32_t best = 0;
    double best_dist = std::fabs(lut[0].a_bps - a_bar);
    for (uint32_t q = 1; q < points; ++q) {
        const double dist = std::fabs(lut[q].a_bps - a_bar);
        if (dist < best_dist) {            // strict: the lower sample wins a tie
            best = q;
            best_dist = dist;
        }
    }
    *tau_out = lut[best].tau;
    *delta_out = lut[best].delta;
    return DECO_OK;
}
