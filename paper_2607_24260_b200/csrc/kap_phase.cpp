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

// kap_fallback_decide: which sequences keep their plan and which take full-context access
// (Section 3.2 "Runtime stability and fallback"; Section 4.2: observed acceptance and profiled
// costs decide when the phase slack of Eq. 13 has turned unfavourable).
extern "C" kap_status kap_fallback_decide(
    int32_t batch, const int64_t* accepted_sum, const int64_t* proposed_sum, int64_t min_proposed,
    double h_prior, const double* s, const double* kv, double w_main, double w_prop, double h_min,
    double s_max, const int32_t* plan_flags, const int32_t* runtime_flags, const double* confidence,
    double confidence_min, uint8_t* force_full, int32_t* reasons, double* h_used, double* slack,
    double* budget_scale)
{
    using kap::fail;
    if (batch < 0) return fail(KAP_ERR_INVALID_ARG, "batch %d", batch);
    if (batch == 0) return KAP_OK;
    if (!accepted_sum || !proposed_sum || !s || !kv || !force_full)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer");
    const double scalars[6] = {h_prior, w_main, w_prop, h_min, s_max, confidence_min};
    for (double x : scalars)
        if (std::isnan(x)) return fail(KAP_ERR_INVALID_ARG, "NaN parameter");
    if (h_prior < 0.0 || h_prior > 1.0 || w_main < 0.0 || w_prop < 0.0 || !std::isfinite(w_main) || !std::isfinite(w_prop))
        return fail(KAP_ERR_INVALID_ARG, "0 <= h_prior <= 1 and finite non-negative weight costs are required");
    for (int32_t b = 0; b < batch; ++b) {
        if (accepted_sum[b] < 0 || proposed_sum[b] < accepted_sum[b])
            return fail(KAP_ERR_INVALID_ARG, "sequence %d: %lld accepted of %lld proposed", b,
                        (long long)accepted_sum[b], (long long)proposed_sum[b]);
        if (!(s[b] >= 0.0) || !(kv[b] >= 0.0) || !std::isfinite(s[b]) || !std::isfinite(kv[b]))
            return fail(KAP_ERR_INVALID_ARG, "sequence %d: s and kv must be finite and non-negative", b);
        if (confidence && std::isnan(confidence[b])) return fail(KAP_ERR_INVALID_ARG, "sequence %d: NaN confidence", b);
    }
    const int64_t need = min_proposed > 1 ? min_proposed : 1;
    for (int32_t b = 0; b < batch; ++b) {
        // Eq. 5 on the running counts; the prior stands in until enough proposals were verified
        const double h = proposed_sum[b] >= need ? (double)accepted_sum[b] / (double)proposed_sum[b] : h_prior;
        const double full = w_main + kv[b], kept = s[b] * kv[b];
        const double delta = h * full - (w_prop + kept);                    // Eq. 13
        const double room = h * full - w_prop;                              // what s * KV may cost at break-even
        double scale;
        if (kept > 0.0) scale = (room > 0.0 ? room : 0.0) / kept;
        else scale = room > 0.0 ? std::numeric_limits<double>::infinity() : 0.0;
        int32_t why = 0;
        const int32_t rt = runtime_flags ? runtime_flags[b] : 0;
        if (rt & KAP_RUNTIME_OVER_CAPACITY) why |= KAP_FALLBACK_CAPACITY;
        if (rt & KAP_RUNTIME_UNSTABLE_METADATA) why |= KAP_FALLBACK_METADATA;
        if (confidence && confidence[b] < confidence_min) why |= KAP_FALLBACK_CONFIDENCE;
        if (s[b] > s_max || (plan_flags && (plan_flags[b] & KAP_PLAN_S_HIGH))) why |= KAP_FALLBACK_S_HIGH;
        if (h < h_min) why |= KAP_FALLBACK_H_LOW;
        if (h <= s[b]) why |= KAP_FALLBACK_NO_MARGIN;                       // Eq. 11
        if (!(delta > 0.0)) why |= KAP_FALLBACK_SLACK;                      // Eq. 8 / Eq. 13
        force_full[b] = why ? 1 : 0;
        if (reasons) reasons[b] = why;
        if (h_used) h_used[b] = h;
        if (slack) slack[b] = delta;
        if (budget_scale) budget_scale[b] = scale;
    }
    return KAP_OK;
}
