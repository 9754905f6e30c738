// kap_compile_plan: Algorithm 1 of the KAP paper from "token spans" onward (Section 3.1,
// "Evidence-to-runtime compilation" / "Selected-KV view materialization"): budgeted selection over
// ranked evidence spans, resolution of the selected tokens to KV pages, logical page indices kept
// for masking, physical pages through the block table.  Host code; touches no GPU.
//
// Representation: the selected token set is kept as a sorted vector of disjoint half-open
// intervals.  A candidate span's cost is its length minus its overlap with that union; taking it
// splices it into the vector.  Pages are emitted by walking the intervals once.
#include <algorithm>
#include <cmath>
#include <cstring>
#include <vector>

#include "kap_internal.h"

namespace kap {

namespace {
thread_local char g_error[512] = "";
}

kap_status fail(kap_status st, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_error, sizeof g_error, fmt, ap);
    va_end(ap);
    return st;
}

const char* last_error_text() { return g_error; }

namespace {

struct Interval { int32_t lo, hi; };   // [lo, hi)

// tokens of [lo, hi) not yet covered by the sorted disjoint `u`
int64_t uncovered(const std::vector<Interval>& u, int32_t lo, int32_t hi) {
    int64_t covered = 0;
    auto it = std::lower_bound(u.begin(), u.end(), lo,
                               [](const Interval& a, int32_t v) { return a.hi <= v; });
    for (; it != u.end() && it->lo < hi; ++it)
        covered += std::min(hi, it->hi) - std::max(lo, it->lo);
    return (int64_t)(hi - lo) - covered;
}

// u := u union [lo, hi), keeping u sorted and disjoint (touching intervals are merged)
void splice(std::vector<Interval>& u, int32_t lo, int32_t hi) {
    if (hi <= lo) return;
    auto first = std::lower_bound(u.begin(), u.end(), lo,
                                  [](const Interval& a, int32_t v) { return a.hi < v; });
    auto last = first;
    while (last != u.end() && last->lo <= hi) {
        lo = std::min(lo, last->lo);
        hi = std::max(hi, last->hi);
        ++last;
    }
    first = u.erase(first, last);
    u.insert(first, Interval{lo, hi});
}

struct Candidate { float score; int32_t lo, hi, index; };

}  // namespace
}  // namespace kap

extern "C" const char* kap_last_error(void) { return kap::last_error_text(); }

extern "C" const char* kap_version(void) { return "kap-b200 0.1 sm_100a"; }

extern "C" kap_status kap_compile_plan(
    int32_t batch, int32_t page_size, const int32_t* ctx_len, const int32_t* span_indptr,
    const int32_t* span_start, const int32_t* span_len, const float* span_score,
    const int32_t* budget_tokens, const int32_t* n_sink, const int32_t* n_recent,
    const uint8_t* force_full, float s_max, const int32_t* bt_indptr, const int32_t* bt_pages,
    int64_t plan_capacity, int32_t* plan_indptr, int32_t* plan_logical_pages,
    int32_t* plan_phys_pages, int32_t* plan_flags, int32_t* selected_tokens,
    uint16_t* plan_token_masks)
{
    using namespace kap;
    if (batch < 0) return fail(KAP_ERR_INVALID_ARG, "batch %d < 0", batch);
    if (page_size <= 0) return fail(KAP_ERR_INVALID_ARG, "page_size %d <= 0", page_size);
    if (!plan_indptr || !plan_flags || (!plan_logical_pages && plan_capacity > 0))
        return fail(KAP_ERR_INVALID_ARG, "NULL output pointer");
    if (batch > 0 && (!ctx_len || !span_indptr || !budget_tokens || !n_sink || !n_recent))
        return fail(KAP_ERR_INVALID_ARG, "NULL input pointer");
    if ((bt_indptr == nullptr) != (bt_pages == nullptr))
        return fail(KAP_ERR_INVALID_ARG, "block table needs both bt_indptr and bt_pages");
    if (plan_phys_pages && !bt_indptr)
        return fail(KAP_ERR_INVALID_ARG, "plan_phys_pages requested without a block table");
    if (plan_token_masks && page_size > 16)
        return fail(KAP_ERR_UNSUPPORTED, "token masks hold 16 bits per page, page_size is %d", page_size);
    if (std::isnan(s_max)) return fail(KAP_ERR_INVALID_ARG, "s_max is NaN");
    if (batch > 0 && span_indptr[0] != 0)
        return fail(KAP_ERR_INVALID_ARG, "span_indptr[0] = %d, expected 0", span_indptr[0]);

    // ---- validation pass: nothing is written unless every sequence is well formed
    for (int32_t b = 0; b < batch; ++b) {
        if (ctx_len[b] <= 0) return fail(KAP_ERR_INVALID_ARG, "ctx_len[%d] = %d <= 0", b, ctx_len[b]);
        if (budget_tokens[b] < 0 || n_sink[b] < 0 || n_recent[b] < 0)
            return fail(KAP_ERR_INVALID_ARG, "negative budget / sink / recent for sequence %d", b);
        if (span_indptr[b + 1] < span_indptr[b])
            return fail(KAP_ERR_INVALID_ARG, "span_indptr decreases at %d", b);
        if (span_indptr[b + 1] > span_indptr[b] && (!span_start || !span_len || !span_score))
            return fail(KAP_ERR_INVALID_ARG, "NULL span arrays");
        for (int32_t i = span_indptr[b]; i < span_indptr[b + 1]; ++i) {
            if (span_len[i] < 0) return fail(KAP_ERR_INVALID_ARG, "span %d has negative length", i);
            if (std::isnan(span_score[i])) return fail(KAP_ERR_INVALID_ARG, "span %d score is NaN", i);
        }
        if (bt_indptr) {
            const int64_t n_pages = ((int64_t)ctx_len[b] + page_size - 1) / page_size;
            if ((int64_t)bt_indptr[b + 1] - bt_indptr[b] < n_pages)
                return fail(KAP_ERR_INVALID_ARG, "block table of sequence %d shorter than %lld pages",
                            b, (long long)n_pages);
            for (int64_t p = 0; p < n_pages; ++p)
                if (bt_pages[bt_indptr[b] + p] < 0)
                    return fail(KAP_ERR_INVALID_ARG, "negative physical page in block table %d", b);
        }
    }

    // ---- selection pass, into temporaries
    std::vector<int32_t> indptr(batch + 1, 0), flags(batch, 0), used_tokens(batch, 0);
    std::vector<int32_t> logical;
    std::vector<uint16_t> masks;
    std::vector<Interval> u;
    std::vector<Candidate> cand;
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t L = ctx_len[b];
        const int32_t n_pages = (int32_t)(((int64_t)L + page_size - 1) / page_size);
        u.clear();
        int64_t used = 0;
        int32_t fl = 0;
        if (force_full && force_full[b]) {
            u.push_back({0, L});
            used = L;
            fl |= KAP_PLAN_FULL;
        } else {
            splice(u, 0, std::min(n_sink[b], L));
            splice(u, std::max<int64_t>(0, (int64_t)L - n_recent[b]), L);
            splice(u, L - 1, L);
            for (const auto& iv : u) used += iv.hi - iv.lo;
            if (used > budget_tokens[b]) {
                fl |= KAP_PLAN_OVER_BUDGET;
            } else {
                cand.clear();
                for (int32_t i = span_indptr[b]; i < span_indptr[b + 1]; ++i) {
                    const int64_t lo = std::max<int64_t>(0, span_start[i]);
                    const int64_t hi = std::min<int64_t>(L, (int64_t)span_start[i] + span_len[i]);
                    if (hi > lo) cand.push_back({span_score[i], (int32_t)lo, (int32_t)hi, i});
                }
                std::sort(cand.begin(), cand.end(), [](const Candidate& a, const Candidate& c) {
                    if (a.score != c.score) return a.score > c.score;
                    if (a.lo != c.lo) return a.lo < c.lo;
                    return a.index < c.index;
                });
                for (const auto& c : cand) {
                    const int64_t fresh = uncovered(u, c.lo, c.hi);
                    if (used + fresh <= budget_tokens[b]) {
                        splice(u, c.lo, c.hi);
                        used += fresh;
                    }
                }
            }
        }
        // pages touched by the union, ascending and unique
        int32_t last_page = -1, n_sel = 0;
        for (const auto& iv : u) {
            const int32_t p0 = std::max(last_page + 1, iv.lo / page_size);
            const int32_t p1 = (iv.hi - 1) / page_size;
            for (int32_t p = p0; p <= p1; ++p) { logical.push_back(p); ++n_sel; }
            last_page = std::max(last_page, p1);
        }
        if (plan_token_masks) {
            // bit t of a listed page: token page*P + t lies in the union (intervals and pages both
            // ascend, so one forward sweep pairs them up)
            masks.resize(logical.size(), 0);
            size_t e = (size_t)indptr[b];
            for (const auto& iv : u) {
                while ((int64_t)logical[e] * page_size + page_size <= iv.lo) ++e;
                for (size_t k = e; k < logical.size() && (int64_t)logical[k] * page_size < iv.hi; ++k) {
                    const int64_t base = (int64_t)logical[k] * page_size;
                    const int lo = (int)std::max<int64_t>(iv.lo - base, 0);
                    const int hi = (int)std::min<int64_t>(iv.hi - base, page_size);
                    masks[k] |= (uint16_t)(((1u << hi) - 1u) & ~((1u << lo) - 1u));
                }
            }
        }
        if ((double)n_sel / (double)n_pages > (double)s_max) fl |= KAP_PLAN_S_HIGH;
        if ((int64_t)logical.size() > (int64_t)INT32_MAX)
            return fail(KAP_ERR_CAPACITY, "plan exceeds 2^31 pages");
        indptr[b + 1] = (int32_t)logical.size();
        flags[b] = fl;
        used_tokens[b] = (int32_t)used;
    }
    if ((int64_t)logical.size() > plan_capacity)
        return fail(KAP_ERR_CAPACITY, "plan needs %lld page entries, capacity is %lld",
                    (long long)logical.size(), (long long)plan_capacity);

    // ---- commit
    std::memcpy(plan_indptr, indptr.data(), sizeof(int32_t) * (size_t)(batch + 1));
    if (!logical.empty())
        std::memcpy(plan_logical_pages, logical.data(), sizeof(int32_t) * logical.size());
    if (plan_phys_pages)
        for (int32_t b = 0; b < batch; ++b)
            for (int32_t i = indptr[b]; i < indptr[b + 1]; ++i)
                plan_phys_pages[i] = bt_pages[bt_indptr[b] + logical[i]];
    if (plan_token_masks && !masks.empty())
        std::memcpy(plan_token_masks, masks.data(), sizeof(uint16_t) * masks.size());
    for (int32_t b = 0; b < batch; ++b) {
        plan_flags[b] = flags[b];
        if (selected_tokens) selected_tokens[b] = used_tokens[b];
    }
    return KAP_OK;
}
