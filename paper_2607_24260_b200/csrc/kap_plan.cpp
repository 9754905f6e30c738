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

// pages touched by sorted disjoint intervals, ascending and unique; appended to `out` when given
int32_t pages_of(const std::vector<Interval>& iv, int32_t page_size, std::vector<int32_t>* out) {
    int32_t last_page = -1, n = 0;
    for (const auto& x : iv) {
        const int32_t p0 = std::max(last_page + 1, x.lo / page_size);
        const int32_t p1 = (x.hi - 1) / page_size;
        for (int32_t p = p0; p <= p1; ++p) { if (out) out->push_back(p); ++n; }
        last_page = std::max(last_page, p1);
    }
    return n;
}

// Growing plans (kap_compile_growing_plan): the emitted list is the part of the plan that does not
// move with the context length (sink + selected spans, or the whole prefix for a full plan),
// followed by reserved entries that kap_refresh_recent fills from the current length.
struct GrowOpts {
    int32_t max_growth;
    int32_t* tail_desc;      // [batch][3] = reserved entries, window tokens, first token they may cover
};

kap_status compile_impl(
    int32_t batch, int32_t page_size, const int32_t* ctx_len, const int32_t* span_indptr,
    const int32_t* span_start, const int32_t* span_len, const float* span_score,
    const int32_t* budget_tokens, const int32_t* n_sink, const int32_t* n_recent,
    const uint8_t* force_full, float s_max, const int32_t* bt_indptr, const int32_t* bt_pages,
    int64_t plan_capacity, int32_t* plan_indptr, int32_t* plan_logical_pages,
    int32_t* plan_phys_pages, int32_t* plan_flags, int32_t* selected_tokens,
    uint16_t* plan_token_masks, const GrowOpts* grow);

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
    return kap::compile_impl(batch, page_size, ctx_len, span_indptr, span_start, span_len, span_score,
                             budget_tokens, n_sink, n_recent, force_full, s_max, bt_indptr, bt_pages,
                             plan_capacity, plan_indptr, plan_logical_pages, plan_phys_pages,
                             plan_flags, selected_tokens, plan_token_masks, nullptr);
}

extern "C" kap_status kap_compile_growing_plan(
    int32_t batch, int32_t page_size, const int32_t* ctx_len, const int32_t* span_indptr,
    const int32_t* span_start, const int32_t* span_len, const float* span_score,
    const int32_t* budget_tokens, const int32_t* n_sink, const int32_t* n_recent,
    const uint8_t* force_full, float s_max, const int32_t* bt_indptr, const int32_t* bt_pages,
    int32_t max_growth, int64_t plan_capacity, int32_t* plan_indptr, int32_t* plan_logical_pages,
    int32_t* plan_phys_pages, uint16_t* plan_token_masks, int32_t* plan_flags,
    int32_t* selected_tokens, int32_t* tail_desc)
{
    using namespace kap;
    if (max_growth < 0) return fail(KAP_ERR_INVALID_ARG, "max_growth %d < 0", max_growth);
    if (!plan_token_masks || !plan_phys_pages || (batch > 0 && !tail_desc))
        return fail(KAP_ERR_INVALID_ARG, "a growing plan needs plan_phys_pages, plan_token_masks and tail_desc");
    if (!bt_indptr) return fail(KAP_ERR_INVALID_ARG, "a growing plan needs a block table");
    const GrowOpts grow{max_growth, tail_desc};
    return compile_impl(batch, page_size, ctx_len, span_indptr, span_start, span_len, span_score,
                        budget_tokens, n_sink, n_recent, force_full, s_max, bt_indptr, bt_pages,
                        plan_capacity, plan_indptr, plan_logical_pages, plan_phys_pages, plan_flags,
                        selected_tokens, plan_token_masks, &grow);
}

namespace kap {
namespace {

kap_status compile_impl(
    int32_t batch, int32_t page_size, const int32_t* ctx_len, const int32_t* span_indptr,
    const int32_t* span_start, const int32_t* span_len, const float* span_score,
    const int32_t* budget_tokens, const int32_t* n_sink, const int32_t* n_recent,
    const uint8_t* force_full, float s_max, const int32_t* bt_indptr, const int32_t* bt_pages,
    int64_t plan_capacity, int32_t* plan_indptr, int32_t* plan_logical_pages,
    int32_t* plan_phys_pages, int32_t* plan_flags, int32_t* selected_tokens,
    uint16_t* plan_token_masks, const GrowOpts* grow)
{
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
    std::vector<Interval> u, fixed;     // fixed: the part of u that does not move with the length
    std::vector<Candidate> cand;
    std::vector<int32_t> tail(grow ? (size_t)batch * 3 : 0, 0);
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t L = ctx_len[b];
        const int32_t n_pages = (int32_t)(((int64_t)L + page_size - 1) / page_size);
        u.clear();
        fixed.clear();
        int64_t used = 0;
        int32_t fl = 0;
        const int64_t window = std::max(n_recent[b], 1);                // the last token is mandatory
        bool moves = false;               // would another length have changed the selection?
        if (force_full && force_full[b]) {
            u.push_back({0, L});
            if (grow) fixed.push_back({0, L});
            used = L;
            fl |= KAP_PLAN_FULL;
        } else {
            if (grow) {
                splice(fixed, 0, std::min(n_sink[b], L));
                moves = (int64_t)n_sink[b] > (int64_t)L - window;
            }
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
                    // a span that reaches the recent window (or past the end) costs a different
                    // number of tokens at another length
                    if (grow && span_len[i] > 0 &&
                        (int64_t)span_start[i] + span_len[i] > std::max<int64_t>(0, (int64_t)L - window))
                        moves = true;
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
                        if (grow) splice(fixed, c.lo, c.hi);
                        used += fresh;
                    }
                }
            }
        }
        // pages touched by the union, ascending and unique
        const int32_t n_sel = pages_of(u, page_size, grow ? nullptr : &logical);
        const std::vector<Interval>& listed = grow ? fixed : u;
        if (grow) pages_of(fixed, page_size, &logical);
        if (plan_token_masks) {
            // bit t of a listed page: token page*P + t lies in the union (intervals and pages both
            // ascend, so one forward sweep pairs them up)
            masks.resize(logical.size(), 0);
            size_t e = (size_t)indptr[b];
            for (const auto& iv : listed) {
                while ((int64_t)logical[e] * page_size + page_size <= iv.lo) ++e;
                for (size_t k = e; k < logical.size() && (int64_t)logical[k] * page_size < iv.hi; ++k) {
                    const int64_t base = (int64_t)logical[k] * page_size;
                    const int lo = (int)std::max<int64_t>(iv.lo - base, 0);
                    const int hi = (int)std::min<int64_t>(iv.hi - base, page_size);
                    masks[k] |= (uint16_t)(((1u << hi) - 1u) & ~((1u << lo) - 1u));
                }
            }
        }
        if (grow) {
            // reserved entries for the window [L' - window, L') at any later length L' (for a full
            // plan: for every token from L on, up to max_growth of them); empty until refreshed
            const bool full = (fl & KAP_PLAN_FULL) != 0;
            int64_t reserve;
            if (full)
                reserve = grow->max_growth == 0 ? 0
                        : ((int64_t)L + grow->max_growth - 1) / page_size - L / page_size + 1;
            else
                reserve = (window + page_size - 2) / page_size + 1;
            for (int64_t r = 0; r < reserve; ++r) logical.push_back(0);
            masks.resize(logical.size(), 0);
            tail[(size_t)b * 3 + 0] = (int32_t)reserve;
            tail[(size_t)b * 3 + 1] = full ? INT32_MAX : (int32_t)window;
            tail[(size_t)b * 3 + 2] = full ? L : 0;
            if (moves) fl |= KAP_PLAN_MOVES_WITH_LENGTH;
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
    if (grow && batch > 0) std::memcpy(grow->tail_desc, tail.data(), sizeof(int32_t) * tail.size());
    return KAP_OK;
}

}  // namespace
}  // namespace kap
