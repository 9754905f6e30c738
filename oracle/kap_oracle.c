/*
 * kap_oracle.c - plain, slow, double-precision CPU statement of what the KAP hot path computes.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the yardstick the CUDA library is checked against; it
 * shares no code, header, table or helper with that library and must never be called from the
 * product path.  Only the test-suite, the smoke check and the benchmark's CPU-baseline leg use it.
 *
 * What it states (sections/algorithms refer to the KAP / GraphSpec paper):
 *
 *   kap_oracle_compile_plan        Algorithm 1, steps SelectEvidenceUnderBudget,
 *                                  ResolveSelectedKVObjects, PreserveLogicalPositions and
 *                                  BuildBlockTable (Section 3.1, "Evidence-to-runtime
 *                                  compilation" and "Selected-KV view materialization"): ranked
 *                                  token spans + a token budget -> the ascending list of logical
 *                                  KV pages the proposal path may see, and their physical pages.
 *                                  This is a heuristic, so the oracle is the algorithm, step by
 *                                  step, on a boolean array with one entry per token.
 *   kap_oracle_selected_decode_attn Section 3.2, "Selected-KV proposal": one query row per
 *                                  sequence (q_prop = 1) at the sequence's last logical position,
 *                                  softmax attention restricted to the tokens of the plan's pages.
 *   kap_oracle_verify_attn         Section 3.2, "Full-context verification": n_q contiguous query
 *                                  rows over the whole block table, row j at logical position
 *                                  L - n_q + j, causal among the rows.
 *   Both attention functions are the textbook definition
 *        out = sum_t softmax_t(scale * <q, k_t>) v_t,   lse = ln sum_t exp(scale * <q, k_t>)
 *   written out with a two-pass, max-subtracted softmax in double precision over bf16 inputs that
 *   are widened exactly.  No blocking, no splitting, no online rescaling.
 *
 * Readings of points the paper leaves open (the same list is kept in the design notes):
 *   - the budget counts tokens of the union of selected positions; sink prefix, recent suffix and
 *     the last token are mandatory and count toward it;
 *   - spans are atomic: one that does not fit is skipped and the scan continues (first fit);
 *   - order: score descending, then clipped start ascending, then input index ascending;
 *   - overlapping spans cost only their new tokens; spans are clipped to [0, L);
 *   - visibility is page-granular: a page with one selected token is visible as a whole;
 *   - the page list is ascending in logical page index.
 * Versus the authors' unpublished implementation these tie-breaks are "parity unpinned"; the
 * attention functions are pinned by definition, closed forms and a dense numpy brute force.
 *
 * KV pool layout (one layer): pool[page][0=K,1=V][kv_head][token_in_page][d], bf16.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

enum { ORC_OK = 0, ORC_INVALID = 1, ORC_CAPACITY = 2 };
enum { ORC_PLAN_FULL = 1, ORC_PLAN_OVER_BUDGET = 2, ORC_PLAN_S_HIGH = 4 };

static double bf16_to_double(uint16_t b) {
    uint32_t u = ((uint32_t)b) << 16;
    float f;
    memcpy(&f, &u, sizeof f);
    return (double)f;
}

/* ------------------------------------------------------------------ plan compilation (Alg. 1) */

typedef struct { int32_t start, end, index; float score; } orc_span;

/* rank order: score descending, clipped start ascending, input index ascending */
static int span_before(const orc_span* a, const orc_span* b) {
    if (a->score != b->score) return a->score > b->score;
    if (a->start != b->start) return a->start < b->start;
    return a->index < b->index;
}

int kap_oracle_compile_plan(
    int32_t batch, int32_t page_size, const int32_t* ctx_len,
    const int32_t* span_indptr, const int32_t* span_start, const int32_t* span_len,
    const float* span_score, const int32_t* budget_tokens, const int32_t* n_sink,
    const int32_t* n_recent, const uint8_t* force_full, float s_max,
    const int32_t* bt_indptr, const int32_t* bt_pages, int64_t plan_capacity,
    int32_t* plan_indptr, int32_t* plan_logical_pages, int32_t* plan_phys_pages,
    int32_t* plan_flags, int32_t* selected_tokens, uint16_t* plan_token_masks)
{
    if (batch < 0 || page_size <= 0) return ORC_INVALID;
    if (plan_token_masks && page_size > 16) return ORC_INVALID;   /* one bit per token of a page */
    /* validate everything first so that outputs stay untouched on error */
    for (int32_t b = 0; b < batch; ++b) {
        if (ctx_len[b] <= 0 || budget_tokens[b] < 0 || n_sink[b] < 0 || n_recent[b] < 0)
            return ORC_INVALID;
        if (span_indptr[b + 1] < span_indptr[b]) return ORC_INVALID;
        for (int32_t i = span_indptr[b]; i < span_indptr[b + 1]; ++i)
            if (span_len[i] < 0 || span_score[i] != span_score[i]) return ORC_INVALID;
        if (bt_indptr) {
            int32_t n_pages = (ctx_len[b] + page_size - 1) / page_size;
            if (bt_indptr[b + 1] - bt_indptr[b] < n_pages) return ORC_INVALID;
        }
    }
    if (span_indptr[0] != 0) return ORC_INVALID;

    int64_t written = 0;
    int32_t* indptr_tmp = (int32_t*)malloc(sizeof(int32_t) * (size_t)(batch + 1));
    int32_t* flags_tmp = (int32_t*)malloc(sizeof(int32_t) * (size_t)(batch + 1));
    int32_t* used_tmp = (int32_t*)malloc(sizeof(int32_t) * (size_t)(batch + 1));
    uint8_t** page_sel = (uint8_t**)calloc((size_t)batch + 1, sizeof(uint8_t*));
    uint8_t** tok_sel = (uint8_t**)calloc((size_t)batch + 1, sizeof(uint8_t*));
    indptr_tmp[0] = 0;
    int rc = ORC_OK;

    for (int32_t b = 0; b < batch; ++b) {
        const int32_t L = ctx_len[b];
        const int32_t n_pages = (L + page_size - 1) / page_size;
        uint8_t* tok = (uint8_t*)calloc((size_t)L, 1);       /* T: one flag per token */
        uint8_t* pg = (uint8_t*)calloc((size_t)n_pages, 1);
        page_sel[b] = pg;
        int32_t flags = 0, used = 0;

        if (force_full && force_full[b]) {
            /* fallback: full-context access (Section 3.2, "Runtime stability and fallback") */
            memset(tok, 1, (size_t)L);
            used = L;
            flags |= ORC_PLAN_FULL;
        } else {
            /* mandatory tokens: sink prefix, recent suffix, the last token */
            for (int32_t t = 0; t < L; ++t) {
                int keep = (t < n_sink[b]) || (t >= L - n_recent[b]) || (t == L - 1);
                if (keep) { tok[t] = 1; ++used; }
            }
            if (used > budget_tokens[b]) {
                flags |= ORC_PLAN_OVER_BUDGET;            /* keep the mandatory set, no spans */
            } else {
                /* clip, drop empties, rank */
                int32_t n_in = span_indptr[b + 1] - span_indptr[b];
                orc_span* sp = (orc_span*)malloc(sizeof(orc_span) * (size_t)(n_in + 1));
                int32_t n = 0;
                for (int32_t i = 0; i < n_in; ++i) {
                    int64_t s0 = span_start[span_indptr[b] + i];
                    int64_t e0 = s0 + (int64_t)span_len[span_indptr[b] + i];
                    if (s0 < 0) s0 = 0;
                    if (e0 > L) e0 = L;
                    if (e0 <= s0) continue;
                    sp[n].start = (int32_t)s0; sp[n].end = (int32_t)e0; sp[n].index = i;
                    sp[n].score = span_score[span_indptr[b] + i];
                    ++n;
                }
                for (int32_t i = 1; i < n; ++i) {             /* insertion sort, rank order */
                    orc_span key = sp[i];
                    int32_t j = i - 1;
                    while (j >= 0 && span_before(&key, &sp[j])) { sp[j + 1] = sp[j]; --j; }
                    sp[j + 1] = key;
                }
                /* greedy first fit over whole spans: a span costs its not-yet-selected tokens */
                for (int32_t i = 0; i < n; ++i) {
                    int32_t fresh = 0;
                    for (int32_t t = sp[i].start; t < sp[i].end; ++t) fresh += !tok[t];
                    if (used + fresh <= budget_tokens[b]) {
                        for (int32_t t = sp[i].start; t < sp[i].end; ++t) tok[t] = 1;
                        used += fresh;
                    }
                }
                free(sp);
            }
        }
        /* resolve tokens to pages: a page is selected iff it holds a selected token */
        int32_t n_sel = 0;
        for (int32_t t = 0; t < L; ++t) if (tok[t]) pg[t / page_size] = 1;
        for (int32_t p = 0; p < n_pages; ++p) n_sel += pg[p];
        if ((double)n_sel / (double)n_pages > (double)s_max) flags |= ORC_PLAN_S_HIGH;
        written += n_sel;
        indptr_tmp[b + 1] = (int32_t)written;
        flags_tmp[b] = flags;
        used_tmp[b] = used;
        tok_sel[b] = tok;
    }
    if (written > plan_capacity) rc = ORC_CAPACITY;
    if (rc == ORC_OK) {
        for (int32_t b = 0; b < batch; ++b) {
            const int32_t n_pages = (ctx_len[b] + page_size - 1) / page_size;
            int64_t o = indptr_tmp[b];
            for (int32_t p = 0; p < n_pages; ++p) {
                if (!page_sel[b][p]) continue;
                plan_logical_pages[o] = p;
                if (plan_phys_pages && bt_indptr) plan_phys_pages[o] = bt_pages[bt_indptr[b] + p];
                if (plan_token_masks) {                       /* bit t: token p*P + t is selected */
                    uint16_t m = 0;
                    for (int32_t t = 0; t < page_size && p * page_size + t < ctx_len[b]; ++t)
                        if (tok_sel[b][p * page_size + t]) m |= (uint16_t)(1u << t);
                    plan_token_masks[o] = m;
                }
                ++o;
            }
            plan_flags[b] = flags_tmp[b];
            if (selected_tokens) selected_tokens[b] = used_tmp[b];
        }
        memcpy(plan_indptr, indptr_tmp, sizeof(int32_t) * (size_t)(batch + 1));
    }
    for (int32_t b = 0; b < batch; ++b) { free(page_sel[b]); free(tok_sel[b]); }
    free(page_sel); free(tok_sel); free(indptr_tmp); free(flags_tmp); free(used_tmp);
    return rc;
}

/* --------------------------------------------------------------------------- masked attention */

/* One query row against the visible tokens of a page list.  q: d doubles.  Visible: every token
 * of every listed page whose logical position t satisfies t <= pos.  Returns the number of
 * visible tokens; out[d], *lse and *wsum (sum of the normalised weights) are written. */
static int64_t attend_row(
    const double* q, const uint16_t* pool, int32_t n_list, const int32_t* list_phys,
    const int32_t* list_logical, const uint16_t* list_masks, int32_t pos, int32_t kv_head, int32_t Hkv,
    int32_t d, int32_t P,
    double scale, double* logits, double* out, double* lse, double* wsum)
{
    const int64_t page_stride = (int64_t)2 * Hkv * P * d;
    int64_t n_vis = 0;
    double zmax = -INFINITY;
    /* pass 1: logits of the visible tokens, and their maximum */
    for (int32_t i = 0; i < n_list; ++i) {
        const int32_t logical = list_logical ? list_logical[i] : i;
        const uint16_t* kpage = pool + (int64_t)list_phys[i] * page_stride
                                     + ((int64_t)0 * Hkv + kv_head) * P * d;
        for (int32_t s = 0; s < P; ++s) {
            const int64_t t = (int64_t)logical * P + s;
            if (t > pos) continue;
            if (list_masks && !((list_masks[i] >> s) & 1)) continue;   /* token-granular visibility */
            double dot = 0.0;
            for (int32_t c = 0; c < d; ++c) dot += q[c] * bf16_to_double(kpage[(int64_t)s * d + c]);
            const double z = scale * dot;
            logits[n_vis++] = z;
            if (z > zmax) zmax = z;
        }
    }
    /* pass 2: weights, normaliser, weighted sum of the value rows */
    for (int32_t c = 0; c < d; ++c) out[c] = 0.0;
    double denom = 0.0;
    int64_t k = 0;
    for (int32_t i = 0; i < n_list; ++i) {
        const int32_t logical = list_logical ? list_logical[i] : i;
        const uint16_t* vpage = pool + (int64_t)list_phys[i] * page_stride
                                     + ((int64_t)1 * Hkv + kv_head) * P * d;
        for (int32_t s = 0; s < P; ++s) {
            const int64_t t = (int64_t)logical * P + s;
            if (t > pos) continue;
            if (list_masks && !((list_masks[i] >> s) & 1)) continue;
            const double w = exp(logits[k++] - zmax);
            denom += w;
            for (int32_t c = 0; c < d; ++c) out[c] += w * bf16_to_double(vpage[(int64_t)s * d + c]);
        }
    }
    double total = 0.0;
    if (n_vis > 0) {
        for (int32_t c = 0; c < d; ++c) out[c] /= denom;
        for (int64_t i = 0; i < n_vis; ++i) total += exp(logits[i] - zmax) / denom;
        *lse = zmax + log(denom);
    } else {
        *lse = -INFINITY;
    }
    if (wsum) *wsum = total;
    return n_vis;
}

/* Shared driver: rows of sequence b are q rows q_indptr[b] .. q_indptr[b+1]-1 (one row per
 * sequence when q_indptr is NULL); row j sits at logical position ctx_len[b] - n_q + j. */
static int attention(
    const uint16_t* q, const int32_t* q_indptr, const uint16_t* pool, int64_t num_pool_pages,
    const int32_t* list_indptr, const int32_t* list_phys, const int32_t* list_logical,
    const uint16_t* list_masks, const int32_t* ctx_len, int32_t batch, int32_t Hq, int32_t Hkv, int32_t d, int32_t P,
    double scale, double* out, double* lse, double* wsum, int64_t* n_visible)
{
    if (batch < 0 || Hq <= 0 || Hkv <= 0 || Hq % Hkv || d <= 0 || P <= 0) return ORC_INVALID;
    const int32_t G = Hq / Hkv;
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t nq = q_indptr ? q_indptr[b + 1] - q_indptr[b] : 1;
        if (ctx_len[b] <= 0 || nq < 0 || nq > ctx_len[b]) return ORC_INVALID;
        if (list_indptr[b + 1] < list_indptr[b]) return ORC_INVALID;
        for (int32_t i = list_indptr[b]; i < list_indptr[b + 1]; ++i) {
            if (list_phys[i] < 0 || list_phys[i] >= num_pool_pages) return ORC_INVALID;
            const int32_t lg = list_logical ? list_logical[i] : i - list_indptr[b];
            if (lg < 0 || (int64_t)lg * P >= ctx_len[b]) return ORC_INVALID;
        }
    }
    int failed = 0;
#ifdef _OPENMP
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
#endif
    for (int32_t b = 0; b < batch; ++b) {
        for (int32_t h = 0; h < Hq; ++h) {
            const int32_t row0 = q_indptr ? q_indptr[b] : b;
            const int32_t nq = q_indptr ? q_indptr[b + 1] - q_indptr[b] : 1;
            const int32_t n_list = list_indptr[b + 1] - list_indptr[b];
            double* logits = (double*)malloc(sizeof(double) * ((size_t)n_list * P + 1));
            double* qd = (double*)malloc(sizeof(double) * (size_t)d);
            if (!logits || !qd) { failed = 1; free(logits); free(qd); continue; }
            for (int32_t j = 0; j < nq; ++j) {
                const int64_t row = row0 + j;
                const int32_t pos = ctx_len[b] - nq + j;
                for (int32_t c = 0; c < d; ++c)
                    qd[c] = bf16_to_double(q[(row * Hq + h) * d + c]);
                double w = 0.0, l = 0.0;
                int64_t nv = attend_row(qd, pool, n_list, list_phys + list_indptr[b],
                                        list_logical ? list_logical + list_indptr[b] : NULL,
                                        list_masks ? list_masks + list_indptr[b] : NULL, pos,
                                        h / G, Hkv, d, P, scale, logits,
                                        out + (row * Hq + h) * d, &l, &w);
                if (lse) lse[row * Hq + h] = l;
                if (wsum) wsum[row * Hq + h] = w;
                if (n_visible) n_visible[row * Hq + h] = nv;
            }
            free(logits); free(qd);
        }
    }
    return failed ? ORC_CAPACITY : ORC_OK;
}

/* Section 3.2, "Selected-KV proposal": q is [batch, Hq, d]; the page list is the plan. */
int kap_oracle_selected_decode_attn(
    const uint16_t* q, const uint16_t* pool, int64_t num_pool_pages,
    const int32_t* plan_indptr, const int32_t* plan_phys_pages, const int32_t* plan_logical_pages,
    const uint16_t* plan_token_masks, const int32_t* ctx_len, int32_t batch, int32_t Hq,
    int32_t Hkv, int32_t d, int32_t P,
    double scale, double* out, double* lse, double* wsum, int64_t* n_visible)
{
    if (plan_token_masks && P > 16) return ORC_INVALID;
    return attention(q, NULL, pool, num_pool_pages, plan_indptr, plan_phys_pages,
                     plan_logical_pages, plan_token_masks, ctx_len, batch, Hq, Hkv, d, P, scale,
                     out, lse, wsum, n_visible);
}

/* Section 3.2, "Full-context verification": q is [sum n_q, Hq, d]; the page list is the whole
 * block table, logical page i at list position i; ctx_len counts the n_q rows' own tokens. */
int kap_oracle_verify_attn(
    const uint16_t* q, const int32_t* q_indptr, const uint16_t* pool, int64_t num_pool_pages,
    const int32_t* bt_indptr, const int32_t* bt_pages, const int32_t* ctx_len, int32_t batch,
    int32_t Hq, int32_t Hkv, int32_t d, int32_t P, double scale, double* out, double* lse,
    double* wsum, int64_t* n_visible)
{
    if (!q_indptr) return ORC_INVALID;
    /* the block table may hold more pages than ceil(L / P); only the first ceil(L / P) exist */
    int32_t* indptr = (int32_t*)malloc(sizeof(int32_t) * (size_t)(batch + 1));
    int32_t* pages = NULL;
    int64_t total = 0;
    for (int32_t b = 0; b < batch; ++b) {
        if (ctx_len[b] <= 0) { free(indptr); return ORC_INVALID; }
        const int32_t n_pages = (ctx_len[b] + P - 1) / P;
        if (bt_indptr[b + 1] - bt_indptr[b] < n_pages) { free(indptr); return ORC_INVALID; }
        total += n_pages;
    }
    pages = (int32_t*)malloc(sizeof(int32_t) * (size_t)(total + 1));
    indptr[0] = 0;
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t n_pages = (ctx_len[b] + P - 1) / P;
        memcpy(pages + indptr[b], bt_pages + bt_indptr[b], sizeof(int32_t) * (size_t)n_pages);
        indptr[b + 1] = indptr[b] + n_pages;
    }
    int rc = attention(q, q_indptr, pool, num_pool_pages, indptr, pages, NULL, NULL, ctx_len, batch, Hq,
                       Hkv, d, P, scale, out, lse, wsum, n_visible);
    free(indptr); free(pages);
    return rc;
}

int kap_oracle_num_threads(void) {
#ifdef _OPENMP
    extern int omp_get_max_threads(void);
    return omp_get_max_threads();
#else
    return 1;
#endif
}
