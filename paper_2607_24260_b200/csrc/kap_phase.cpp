// kap_phase_model: the paper's memory-traffic cost model of a propose-k / verify cycle and its
// phase boundary (Section 4.1-4.2, Eqs. 3-15), as a host-side calculator.  Feed it measured times
// (e.g. this library's per-pass attention times as KV terms) or byte counts; the units cancel.
#include <cmath>
#include <limits>

#include "kap_internal.h"

extern "C" kap_status kap_phase_model(double k, double h, double s, double w_main, double w_prop,
                                      double kv, double* out)
{
    using kap::fail;
    if (!out) return fail(KAP_ERR_INVALID_ARG, "NULL output");
    const double v[6] = {k, h, s, w_main, w_prop, kv};
    for (double x : v)
        if (!std::isfinite(x)) return fail(KAP_ERR_INVALID_ARG, "non-finite input");
    if (k < 1.0 || h < 0.0 || h > 1.0 || s < 0.0 || w_main < 0.0 || w_prop < 0.0 || kv < 0.0)
        return fail(KAP_ERR_INVALID_ARG, "k >= 1, 0 <= h <= 1, s >= 0 and non-negative costs are required");
    const double cost_full = w_main + kv;                               // Eq. 3
    const double cost_base = (1.0 + k * h) * cost_full;                 // Eq. 6
    const double cost_plan = k * (w_prop + s * kv) + cost_full;         // Eq. 7
    const double slack = h * cost_full - (w_prop + s * kv);             // Eq. 13
    // break-even KV scale (Eq. 12 in its general form): (h - s) KV = W_prop - h W_main
    double kv_crit;
    const double need = w_prop - h * w_main;
    if (h > s) kv_crit = need > 0.0 ? need / (h - s) : 0.0;
    else kv_crit = need < 0.0 ? 0.0 : std::numeric_limits<double>::infinity();   // h <= s: no KV margin
    out[0] = cost_full;
    out[1] = cost_base;
    out[2] = cost_plan;
    out[3] = cost_plan > 0.0 ? cost_base / cost_plan : std::numeric_limits<double>::infinity();
    out[4] = slack;
    out[5] = kv_crit;
    out[6] = slack > 0.0 ? 1.0 : 0.0;                                   // Eq. 8: plan is beneficial
    out[7] = h - s;                                                     // Eq. 11: margin, must be > 0
    return KAP_OK;
}
