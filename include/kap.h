/*
 * kap.h - C ABI of the B200 (sm_100a) library for the KAP / GraphSpec decode hot path:
 * decode-time attention over the selected-KV view that a runtime access plan defines, and the
 * full-context verification attention that guards it.
 *
 * The three operations come from the KAP paper (Section 2.1, Eq. 1: the runtime access plan
 * A = (U, M, pos, rho_access, rho_verify); Section 3.1, Algorithm 1: the GraphSpec compiler;
 * Section 3.2: the GraphSpec executor's two paths):
 *
 *   kap_compile_plan          Algorithm 1 from "token spans" onward: budgeted selection of ranked
 *                             evidence spans (U), resolution to KV pages and physical pages through
 *                             the block table (M), logical page indices kept (pos), fallback flags.
 *   kap_selected_decode_attn  "Selected-KV proposal": one query row per sequence (q_prop = 1) at
 *                             its full-sequence logical position, attending only to the plan's
 *                             pages of the paged KV pool.
 *   kap_verify_attn           "Full-context verification": n_q contiguous query rows per sequence
 *                             over the whole block table, original logical positions, causal among
 *                             the rows.
 *
 * Conventions
 *   - Plain C, no exceptions, no aborts: every call returns a kap_status; kap_last_error() gives
 *     a thread-local message for the last failure on the calling thread.
 *   - Pointers are marked HOST or DEVICE.  The caller owns every buffer it passes; the library
 *     owns only kap_workspace objects.  A workspace belongs to one device and may be used by one
 *     host thread at a time; different workspaces are independent.
 *   - The attention calls only enqueue kernels on the given CUDA stream and return (asynchronous,
 *     no allocation, no synchronisation; they can be captured into a CUDA graph).  Problems a
 *     kernel detects (a page index outside the pool, a bounded wait that ran out) set a status
 *     word that kap_workspace_check() reads.
 *   - KV pool layout of one layer ("HND"): bf16 pool[page][2][Hkv][P][d], index 0 = K, 1 = V, so the
 *     K (or V) rows of one page and one KV head are P*d contiguous elements.  Supported shape:
 *     d = 128, P = 16, Hq = G*Hkv with G in {1, 2, 4, 8, 16}; anything else is KAP_ERR_UNSUPPORTED.
 *     The pool base address must be 16-byte aligned.
 *   - Keys in the pool are already position-encoded at their logical index and queries arrive
 *     encoded at theirs (the paper's logical-position preservation, Section 2.1); the kernels
 *     apply no positional operation - positions only decide visibility.
 */
#ifndef KAP_H_
#define KAP_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    KAP_OK = 0,
    KAP_ERR_INVALID_ARG = 1,   /* malformed input; outputs untouched */
    KAP_ERR_CAPACITY = 2,      /* result does not fit the caller's buffers / the workspace */
    KAP_ERR_UNSUPPORTED = 3,   /* shape outside the supported set */
    KAP_ERR_CUDA = 4,          /* a CUDA runtime / driver call failed */
    KAP_ERR_TIMEOUT = 5,       /* a bounded device-side wait ran out */
    KAP_ERR_DEVICE_INDEX = 6   /* a kernel met an out-of-range page or list index */
} kap_status;

/* Layout of one layer's paged KV pool.  HND (default): bf16 pool[page][2][Hkv][P][d], the K (or V)
 * rows of one page and one KV head are contiguous.  NHD: bf16 pool[page][2][P][Hkv][d], token-major
 * (what a fused QKV projection writes).  Same page size, same 65 536 bytes per page. */
enum {
    KAP_KV_HND = 0,
    KAP_KV_NHD = 1
};

/* per-sequence plan flags (bit-or) written by kap_compile_plan */
enum {
    KAP_PLAN_FULL = 1,         /* identity plan: the sequence takes full-context access */
    KAP_PLAN_OVER_BUDGET = 2,  /* the mandatory tokens alone exceed the budget; no span selected */
    KAP_PLAN_S_HIGH = 4,       /* retained ratio s (Eq. 4, in pages) > s_max: caller should fall back */
    KAP_PLAN_MOVES_WITH_LENGTH = 8  /* growing plans only: compiled at another length, Algorithm 1
                                       could have selected other spans (see kap_compile_growing_plan) */
};

/*
 * kap_compile_plan - Algorithm 1, steps SelectEvidenceUnderBudget, ResolveSelectedKVObjects,
 * PreserveLogicalPositions, BuildBlockTable (Section 3.1).  HOST pointers in and out; runs on the
 * calling thread; touches no GPU.  Runs once per request (the paper counts it inside TTFT).
 *
 * Per sequence b with L = ctx_len[b] tokens and n_pages = ceil(L / page_size):
 *   1. mandatory tokens: the sink prefix [0, n_sink), the recent suffix [L - n_recent, L) and the
 *      last token L-1.  They count toward the budget.  If they alone exceed budget_tokens[b] the
 *      plan is the mandatory set and KAP_PLAN_OVER_BUDGET is set.
 *   2. spans span_indptr[b] .. span_indptr[b+1]-1 are clipped to [0, L) (empty ones dropped) and
 *      ranked by score descending, then clipped start ascending, then input index ascending.
 *   3. first fit over whole spans: a span is taken iff the tokens it adds to the union fit the
 *      remaining budget; otherwise it is skipped and the scan continues.  Spans are never cut.
 *   4. a logical page is selected iff it holds a selected token; pages are emitted in ascending
 *      logical order; plan_phys_pages[i] = bt_pages[bt_indptr[b] + plan_logical_pages[i]].
 *   5. force_full[b] != 0 selects every page and sets KAP_PLAN_FULL (the fallback path, Section 3.2
 *      "Runtime stability and fallback"); selected/total pages > s_max sets KAP_PLAN_S_HIGH.
 *   6. plan_token_masks (optional, page_size <= 16): one 16-bit word per listed page, bit t set
 *      iff token page * page_size + t belongs to the selected union U.  It is the plan's visibility
 *      mask (Section 3.1 "Selected-KV view materialization") at token granularity; without it the
 *      attention call treats every token of a listed page as visible.
 *
 * plan_indptr[batch+1], plan_flags[batch] and selected_tokens[batch] (may be NULL) are written;
 * plan_logical_pages / plan_phys_pages receive plan_indptr[batch] entries and must hold
 * plan_capacity entries.  plan_phys_pages may be NULL; it requires a block table otherwise.
 * force_full and the block table may be NULL.  plan_token_masks may be NULL; it must hold
 * plan_capacity entries otherwise (KAP_ERR_UNSUPPORTED when page_size > 16).
 *
 * Errors: KAP_ERR_INVALID_ARG for batch < 0, page_size <= 0, ctx_len <= 0, a negative budget /
 * sink / recent / span length, a NaN score, a non-monotone span_indptr, a block table shorter than
 * n_pages, a negative block-table entry, or a required pointer that is NULL; KAP_ERR_CAPACITY when
 * the plan needs more than plan_capacity entries (one of the paper's fallback conditions: a plan
 * larger than the space reserved for it).  On any error no output is written.
 */
kap_status kap_compile_plan(
    int32_t batch, int32_t page_size,
    const int32_t* ctx_len,            /* HOST [batch] tokens in the KV cache incl. the current one */
    const int32_t* span_indptr,        /* HOST [batch+1] */
    const int32_t* span_start,         /* HOST [n_spans] first token of each span */
    const int32_t* span_len,           /* HOST [n_spans] */
    const float* span_score,           /* HOST [n_spans] priority, higher first */
    const int32_t* budget_tokens,      /* HOST [batch] */
    const int32_t* n_sink,             /* HOST [batch] */
    const int32_t* n_recent,           /* HOST [batch] */
    const uint8_t* force_full,         /* HOST [batch] or NULL */
    float s_max,                       /* >= 1 disables the KAP_PLAN_S_HIGH test */
    const int32_t* bt_indptr,          /* HOST [batch+1] CSR block table, or NULL */
    const int32_t* bt_pages,           /* HOST logical page -> physical page */
    int64_t plan_capacity,
    int32_t* plan_indptr,              /* HOST out [batch+1] */
    int32_t* plan_logical_pages,       /* HOST out, ascending per sequence */
    int32_t* plan_phys_pages,          /* HOST out or NULL */
    int32_t* plan_flags,               /* HOST out [batch] */
    int32_t* selected_tokens,          /* HOST out [batch] or NULL: size of the token union */
    uint16_t* plan_token_masks);       /* HOST out or NULL: per listed page, bit t = token t selected */

/*
 * Workspace: the split-K work list of one launch shape and the buffers for the partial results
 * (Section 3.2 "Runtime stability and fallback" asks for a workspace that is reused and for metadata
 * whose shapes do not change between steps).  The paper has no counterpart for the split-K schedule itself; it is how this
 * library spreads one sequence's page list over the GPU's SMs.
 *
 * kap_workspace_create allocates (cudaMalloc / cudaMallocHost) on `device`:
 *   max_items          most work items (CTAs) one schedule may hold
 *   max_rows_per_item  most query rows of one (sequence, KV head): n_q * (Hq / Hkv)
 *   max_batch          most sequences
 * kap_schedule (HOST arrays) splits every (sequence, KV head) page list of list_len[b] pages into
 * near-equal contiguous chunks so that the chunks fill the GPU in whole waves (short lists: a half
 * or a quarter of one, so that a CTA has more than a page or two to stream), uploads the work
 * list on `cuda_stream` (asynchronous copy from pinned memory owned by the workspace) and keeps
 * it until the next kap_schedule.  The schedule depends only on the page counts, so one schedule
 * serves every layer and every step whose list lengths and row counts are unchanged; a call that
 * repeats the previous call's counts and options returns at once and uploads nothing.
 * A workspace serves one attention call at a time: use one for the proposal path and another for
 * the verification path.  max_chunk_pages = 0 picks the default chunk cap.
 * Errors: KAP_ERR_INVALID_ARG (NULL, batch < 0, list_len <= 0, n_q < 1, bad head counts),
 * KAP_ERR_CAPACITY (batch > max_batch; rows or items beyond what the workspace was created for;
 * max_batch > 8191: every CTA stages the batch's offset arrays in shared memory), KAP_ERR_CUDA.
 * A kap_schedule that fails leaves the previous schedule in force, whole.
 * Neither call changes the calling thread's current device (it is switched to the workspace's
 * device inside the call and put back).  The attention calls, by contrast, must be made with the
 * workspace's device current - like any launch on one of its streams - and return
 * KAP_ERR_INVALID_ARG otherwise.
 */
typedef struct kap_workspace kap_workspace;

kap_status kap_workspace_create(kap_workspace** ws, int32_t device, int32_t max_items,
                                int32_t max_rows_per_item, int32_t max_batch);
void kap_workspace_destroy(kap_workspace* ws);

kap_status kap_schedule(
    kap_workspace* ws, int32_t batch,
    const int32_t* list_len,           /* HOST [batch] pages in each sequence's list */
    const int32_t* n_q,                /* HOST [batch] query rows per sequence, NULL => 1 each */
    int32_t num_q_heads, int32_t num_kv_heads,
    int32_t max_chunk_pages,           /* cap on pages per work item, 0 => default */
    void* cuda_stream);

/* The schedule kap_schedule would build for `cta_slots` resident CTAs per wave and clusters of
 * at most `max_cluster` CTAs (resident clusters approximated as cta_slots / size), written to HOST
 * arrays without touching a GPU (for inspection and tests).  items_out holds max_items rows of
 * 8 int32: seq, kv_head, page_begin, page_end (relative to the sequence's list; shared evenly by
 * the CTAs of the item's cluster), group, partial slot, n_splits, n_q; longest chunks first.
 * max_chunk = most pages one CTA streams.  Any output pointer may be NULL.  Like kap_schedule it
 * has no counterpart in the paper.  Errors as kap_schedule, minus KAP_ERR_CUDA. */
kap_status kap_schedule_host(
    int32_t batch, const int32_t* list_len, const int32_t* n_q, int32_t num_q_heads,
    int32_t num_kv_heads, int32_t cta_slots, int32_t max_cluster, int32_t max_chunk_pages,
    int32_t max_items, int32_t* items_out, int32_t* n_items, int32_t* n_merge_groups,
    int32_t* max_chunk, int32_t* cluster_size);

/* what the last kap_schedule produced; any pointer may be NULL */
kap_status kap_schedule_info(const kap_workspace* ws, int32_t* n_items, int32_t* n_merge_groups,
                             int32_t* max_chunk_pages, int32_t* ctas_per_wave,
                             int32_t* cluster_size);

/*
 * kap_workspace_set_kv_layout - layout (KAP_KV_HND, the default, or KAP_KV_NHD) of the pools that
 * later kap_selected_decode_attn / kap_verify_attn calls on this workspace will be given.  The
 * paper does not fix a pool layout; both are read with the same tiles, bytes and arithmetic, and
 * results are identical bit for bit.  Host only, no GPU work.  KAP_ERR_INVALID_ARG for a NULL
 * workspace or an unknown layout.
 */
kap_status kap_workspace_set_kv_layout(kap_workspace* ws, int32_t kv_layout);

/*
 * kap_selected_decode_attn - Section 3.2 "Selected-KV proposal".  For sequence b and query head h
 * (KV head g = h / G), with Vis(b) = the tokens t < ctx_len[b] of the plan's pages:
 *     z_t = sm_scale * <q[b,h,:], K[g,t,:]>,   out[b,h,:] = sum_t softmax_t(z) V[g,t,:],
 *     lse[b,h] = ln sum_t exp(z_t)            (natural log)
 * computed as split-K flash decoding (bf16 tensor-core products, fp32 accumulation, base-2 online
 * softmax); the splits' results are merged by log-sum-exp, inside a thread-block cluster through
 * distributed shared memory and, for lists too long for one cluster, by a separate merge pass.  One layer per call.
 * plan_logical_pages == NULL means "logical page = position in the list" (identity plan).
 * plan_token_masks == NULL means every token of a listed page is visible (page-granular view:
 * the page is read whole either way).  With masks, Vis(b) shrinks to the tokens whose bit is set
 * (still t < ctx_len[b]); masked tokens get weight exactly 0, and a head that sees no token at all
 * returns out = 0 and lse = -inf.  The bytes read do not change.
 * The plan arrays are the DEVICE copies of kap_compile_plan's outputs; `ws` must hold a schedule
 * made from the same per-sequence list lengths with n_q = NULL.
 * Errors: KAP_ERR_INVALID_ARG (NULL pointer, batch mismatch with the schedule, misaligned pool),
 * KAP_ERR_UNSUPPORTED (shape), KAP_ERR_CUDA (launch failure).  Nothing is enqueued on error.
 */
kap_status kap_selected_decode_attn(
    const void* q,                     /* DEVICE bf16 [batch, Hq, d] */
    const void* kv_pool,               /* DEVICE bf16 [num_pool_pages][2][Hkv][P][d], this layer */
    int64_t num_pool_pages,
    const int32_t* plan_indptr,        /* DEVICE [batch+1] */
    const int32_t* plan_phys_pages,    /* DEVICE [plan_indptr[batch]] */
    const int32_t* plan_logical_pages, /* DEVICE same length, or NULL */
    const uint16_t* plan_token_masks,  /* DEVICE same length, or NULL */
    const int32_t* ctx_len,            /* DEVICE [batch] */
    int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t page_size,
    float sm_scale,
    void* out,                         /* DEVICE bf16 [batch, Hq, d] */
    float* lse,                        /* DEVICE fp32 [batch, Hq] or NULL */
    kap_workspace* ws, void* cuda_stream);

/*
 * kap_verify_attn - Section 3.2 "Full-context verification".  Sequence b has n_q = q_indptr[b+1] -
 * q_indptr[b] query rows (the paper's q_verify = k + 1 window, or k rows); row j sits at logical
 * position p_j = ctx_len[b] - n_q + j and sees every token t <= p_j of the full block table
 * (ctx_len counts the rows' own tokens, whose K/V are already in the pool: the verifier advances
 * the full KV state in the same pass).  Same formula, same kernels as the proposal path.
 * bt_pages may list more pages than the schedule's list_len[b] per sequence; only the first
 * list_len[b] are read.  `ws` must hold a schedule made with the same n_q and with
 * list_len[b] >= ceil(ctx_len[b] / P): normally equal, but a schedule made for the longest context
 * a graph-captured loop can reach serves every shorter one - pages at or beyond ctx_len are read
 * (they must be valid pool pages) and contribute nothing.  Errors as kap_selected_decode_attn.
 */
kap_status kap_verify_attn(
    const void* q,                     /* DEVICE bf16 [sum n_q, Hq, d], a sequence's rows contiguous */
    const int32_t* q_indptr,           /* DEVICE [batch+1] */
    const void* kv_pool, int64_t num_pool_pages,
    const int32_t* bt_indptr,          /* DEVICE [batch+1] CSR full block table */
    const int32_t* bt_pages,           /* DEVICE */
    const int32_t* ctx_len,            /* DEVICE [batch] */
    int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t page_size,
    float sm_scale,
    void* out,                         /* DEVICE bf16 [sum n_q, Hq, d] */
    float* lse,                        /* DEVICE fp32 [sum n_q, Hq] or NULL */
    kap_workspace* ws, void* cuda_stream);

/*
 * kap_append_kv - place the K and V rows of newly processed tokens into their physical KV slots
 * (the paper's slot mapping: Section 3.1 "Selected-KV view materialization"; each proposal step and
 * the verifier pass write the K/V of the tokens they process, Section 3.2).  Token j of sequence b
 * goes to logical position ctx_len[b] + j, i.e. page bt_pages[bt_indptr[b] + pos / P], slot
 * pos % P, for both K and V and every KV head.  With advance != 0 the kernel then sets
 * ctx_len[b] += n_new[b] on the device, so that a loop "append -> attention" over several decoding
 * steps can be captured into one CUDA graph.  One CTA per sequence; asynchronous on cuda_stream.
 *
 * Running k proposal steps on one compiled plan: compile the plan for the length the sequence
 * will have at the end of the cycle (ctx_len + k, with the recent window widened by k), and run
 * the attention calls with the current device ctx_len: pages and slots past ctx_len are masked, so
 * tokens that have not been appended yet are never seen.
 *
 * The block table must already hold a page for every position written.  A position without a
 * page, a page outside the pool or a negative ctx_len is reported in *device_status
 * (1 << KAP_ERR_DEVICE_INDEX) and that element is not written.
 * Errors: KAP_ERR_UNSUPPORTED (shape), KAP_ERR_INVALID_ARG (NULL or misaligned pointer),
 * KAP_ERR_CUDA.
 */
kap_status kap_append_kv(
    const void* k_new,                 /* DEVICE bf16 [sum n_new, Hkv, d] */
    const void* v_new,                 /* DEVICE bf16 [sum n_new, Hkv, d] */
    const int32_t* new_indptr,         /* DEVICE [batch+1], or NULL: one new token per sequence */
    void* kv_pool, int64_t num_pool_pages,
    const int32_t* bt_indptr,          /* DEVICE [batch+1] CSR block table */
    const int32_t* bt_pages,           /* DEVICE */
    int32_t* ctx_len,                  /* DEVICE [batch], read; updated when advance != 0 */
    int32_t advance,
    int32_t batch, int32_t num_kv_heads, int32_t head_dim, int32_t page_size,
    int32_t kv_layout,                 /* KAP_KV_HND or KAP_KV_NHD: layout of kv_pool */
    int32_t* device_status,            /* DEVICE int32 or NULL */
    void* cuda_stream);

/*
 * kap_top3_accept - the verifier's tolerant acceptance rule (Section 3.2, Eq. 2: the verifier
 * transition returns the number m of proposed tokens accepted consecutively from the start of the
 * window and the next carry token; the Top-3 rule accepts a proposed token when it is among the
 * target model's three best candidates under the full context).
 *
 * Sequence b owns logits rows row_indptr[b] .. row_indptr[b+1]-1: its verification window of
 * k_b + 1 rows (carry row first).  proposed[r] is the token proposed for the position that row r
 * predicts; the last row of a sequence has no proposal (its entry is ignored).
 *   top3[r][0..2]  the three highest logits of row r: value descending, lower index first on equal
 *                  values, NaN ranked below every number (fp32 comparisons on the fp32 inputs:
 *                  exact, no tolerance).
 *   accepted[b]    m = the largest m <= k_b with proposed[row i] in top3[row i] for all i < m.
 *   next_token[b]  top3[row m][0]: the verifier's own best token at the first position that was not
 *                  accepted, or at the bonus position when all k_b were (the paper leaves the
 *                  choice of the carry open; this is the reading used here).
 *   ctx_len[b]     (optional commit step) reduced by k_b - m: with the proposals' K/V appended
 *                  during the cycle, ctx_len counts all k_b of them on entry and only the accepted
 *                  ones on return; the rejected tokens' slots are overwritten by the next
 *                  cycle's appends.  The carry token is not in the cache yet.
 * A window without any row (row_indptr[b+1] == row_indptr[b]: a sequence that sits this cycle out)
 * has nothing to accept and no row to take a carry from: accepted[b] = 0, next_token[b] = -1,
 * ctx_len[b] unchanged.
 * logits: DEVICE fp32, row r starts at logits + r * row_stride.  All outputs DEVICE int32; top3 is
 * [total_rows, 3] and is required (it is also the scratch between the two kernels).
 * Errors: KAP_ERR_INVALID_ARG (NULL pointer, vocab < 3, row_stride < vocab, negative counts),
 * KAP_ERR_CUDA.  Asynchronous on cuda_stream.
 */
kap_status kap_top3_accept(
    const float* logits, int64_t row_stride,
    const int32_t* row_indptr,         /* DEVICE [batch+1] */
    const int32_t* proposed,           /* DEVICE [total_rows] */
    int32_t batch, int32_t total_rows, int32_t vocab,
    int32_t* top3,                     /* DEVICE out [total_rows, 3] */
    int32_t* accepted,                 /* DEVICE out [batch] */
    int32_t* next_token,               /* DEVICE out [batch] */
    int32_t* ctx_len,                  /* DEVICE in/out [batch], or NULL: no commit */
    void* cuda_stream);

/*
 * kap_phase_model - the paper's cost model of one propose-k / verify cycle and its phase boundary
 * (Section 4.1 and 4.2, Eqs. 3-15).  HOST only; any consistent unit (bytes, seconds).
 *   k        proposed tokens per cycle (>= 1)            h  acceptance rate in [0, 1] (Eq. 5)
 *   s        retained-KV ratio (Eq. 4, >= 0)             kv cost of reading the full KV cache
 *   w_main   weight cost of one main-model step          w_prop  weight cost of one proposal step
 *            (self-speculation: w_prop = w_main)
 * out[8]:  [0] Cost_full = w_main + kv (Eq. 3)           [1] Cost_base = (1 + k h) Cost_full (Eq. 6)
 *          [2] Cost_plan = k (w_prop + s kv) + Cost_full (Eq. 7)
 *          [3] speedup = Cost_base / Cost_plan           [4] phase slack = h Cost_full - (w_prop + s kv) (Eq. 13)
 *          [5] break-even KV: (w_prop - h w_main) / (h - s) when h > s (Eq. 12 in general form; 0 if
 *              already negative), +inf when h <= s and the right-hand side is positive
 *          [6] 1 if the plan lies in the positive-speedup region (slack > 0, Eq. 8), else 0
 *          [7] h - s (Eq. 11)
 * Cost_base - Cost_plan = k * slack, so k never changes the sign (the paper's first implication).
 * Errors: KAP_ERR_INVALID_ARG for NULL out, non-finite input, k < 1, h outside [0, 1], negative
 * s or costs; out is untouched on error.
 */
kap_status kap_phase_model(double k, double h, double s, double w_main, double w_prop, double kv,
                           double* out /* HOST [8] */);

/* runtime conditions the caller reports to kap_fallback_decide (bit-or) */
enum {
    KAP_RUNTIME_OVER_CAPACITY = 1,     /* the plan did not fit the space reserved for it (a compile
                                          or view call returned KAP_ERR_CAPACITY) */
    KAP_RUNTIME_UNSTABLE_METADATA = 2  /* list lengths / shapes changed so that the captured graphs
                                          and the schedule no longer apply */
};
/* why kap_fallback_decide sends a sequence to full-context access (bit-or) */
enum {
    KAP_FALLBACK_CAPACITY = 1, KAP_FALLBACK_METADATA = 2, KAP_FALLBACK_CONFIDENCE = 4,
    KAP_FALLBACK_S_HIGH = 8, KAP_FALLBACK_H_LOW = 16, KAP_FALLBACK_NO_MARGIN = 32,
    KAP_FALLBACK_SLACK = 64
};

/*
 * kap_fallback_decide - the fallback rule of Section 3.2 ("Runtime stability and fallback") with
 * the quantities of Section 4: the executor returns a request to full-context access when its plan
 * exceeds the compact workspace, breaks the metadata-stability assumptions, comes from priors of
 * too little confidence, retains too much KV (s high) or is accepted too rarely (h low); Section 4.2
 * adds that observed acceptance and profiled costs decide when the phase slack has turned
 * unfavourable.  HOST only, per sequence b:
 *   h      = accepted_sum[b] / proposed_sum[b] (Eq. 5; the running sums of kap_top3_accept's
 *            accepted[] and of the proposals verified) once proposed_sum[b] >= max(min_proposed, 1),
 *            h_prior before that
 *   slack  = h (w_main + kv[b]) - (w_prop + s[b] kv[b])                              (Eq. 13)
 *   reasons (bit-or): CAPACITY / METADATA from runtime_flags[b]; CONFIDENCE when confidence[b] <
 *            confidence_min; S_HIGH when s[b] > s_max or plan_flags[b] has KAP_PLAN_S_HIGH;
 *            H_LOW when h < h_min; NO_MARGIN when h <= s[b] (Eq. 11: no context length can make
 *            such a plan pay); SLACK when slack <= 0 (Eq. 8).
 *   force_full[b] = 1 iff any reason applies - feed it to kap_compile_plan's force_full for the
 *            next cycle (the identity plan through the same kernels).
 *   budget_scale[b] = (h (w_main + kv) - w_prop) / (s kv), floored at 0: the factor by which s
 *            could be multiplied before the slack reaches zero - room to widen the budget when
 *            > 1, the cut that would bring the plan back to break-even when < 1 (the paper's
 *            "budget adjustment"; +inf when s kv = 0 and there is room).
 * Costs are in any one unit: bytes, or measured times (attention only: w_main = w_prop = 0,
 * kv[b] = the sequence's share of the measured full-context decode time, s[b] = measured
 * proposal time / full time, or the page ratio kap_compile_plan realised).
 * plan_flags, runtime_flags, confidence, reasons, h_used, slack and budget_scale may be NULL.
 * Errors: KAP_ERR_INVALID_ARG (NULL pointer, negative batch, NaN, h_prior outside [0, 1],
 * negative or non-finite costs, more accepted than proposed); outputs untouched on error.
 */
kap_status kap_fallback_decide(
    int32_t batch,
    const int64_t* accepted_sum,       /* HOST [batch] */
    const int64_t* proposed_sum,       /* HOST [batch] */
    int64_t min_proposed, double h_prior,
    const double* s,                   /* HOST [batch] retained-KV ratio (Eq. 4) */
    const double* kv,                  /* HOST [batch] cost of reading the sequence's whole KV */
    double w_main, double w_prop,
    double h_min, double s_max,
    const int32_t* plan_flags,         /* HOST [batch] KAP_PLAN_* or NULL */
    const int32_t* runtime_flags,      /* HOST [batch] KAP_RUNTIME_* or NULL */
    const double* confidence,          /* HOST [batch] or NULL */
    double confidence_min,
    uint8_t* force_full,               /* HOST out [batch] */
    int32_t* reasons,                  /* HOST out [batch] or NULL */
    double* h_used, double* slack, double* budget_scale);   /* HOST out [batch] or NULL */

/*
 * kap_compile_growing_plan / kap_refresh_recent - one compiled plan for a context that grows
 * (Section 3.2: k proposal steps per cycle, many cycles per request; the plan is compiled once per
 * request, Section 3.1).  The selected union U of Algorithm 1 has a part that does not depend on
 * the length - the sink prefix and the selected spans - and the recent window [L - n_recent, L)
 * (at least the last token), which moves.  kap_compile_growing_plan runs Algorithm 1 exactly as
 * kap_compile_plan does (same arguments, same ranking, same budget accounting at ctx_len) but
 * lists, per sequence, the pages and token masks of the fixed part followed by reserved entries
 * with empty masks; kap_refresh_recent, a small kernel, rewrites the reserved entries from the
 * device-side ctx_len: the window's pages, with masks that omit tokens the fixed part already
 * lists.  kap_selected_decode_attn on these arrays (plan_token_masks is required) then sees
 * exactly fixed part + window at the current length, and one kap_schedule (list lengths never
 * change) serves every step.  A page that holds both fixed and window tokens is listed twice with
 * disjoint masks; a reserved entry that is not needed repeats the sequence's last page with an
 * empty mask (read like any page, contributes nothing).
 *
 * A full-context plan (force_full) lists the whole prefix and reserves entries for every token
 * from ctx_len on, up to max_growth more tokens; for other sequences max_growth is not needed.
 *
 * When is this the plan Algorithm 1 would compile at the longer length?  Whenever the sink and
 * every non-empty span end at or before ctx_len - max(n_recent, 1): then no span shares tokens
 * with the window at this or any greater length and span costs do not change.  Otherwise the
 * sequence gets KAP_PLAN_MOVES_WITH_LENGTH: the arrays are still valid (fixed part + window, no
 * token twice) but a fresh compile could select other spans.
 *
 * tail_desc[b] = { reserved entries, window tokens (INT32_MAX: everything), first token the
 * reserved entries may cover }; copy it to the device for kap_refresh_recent.  selected_tokens and
 * the flags describe the plan at ctx_len.  The reserved entries start out empty: call
 * kap_refresh_recent before the first attention call.
 * Errors of kap_compile_growing_plan: as kap_compile_plan, plus KAP_ERR_INVALID_ARG for
 * max_growth < 0, a missing block table, or a NULL plan_phys_pages / plan_token_masks / tail_desc.
 *
 * kap_refresh_recent: DEVICE pointers; asynchronous on cuda_stream; captured into CUDA graphs
 * like the attention calls.  Problems found on the device (a window page without a block-table
 * entry, a page outside the pool, a context that outgrew the reservation, ctx_len <= 0) set
 * 1 << KAP_ERR_DEVICE_INDEX in *device_status, or in the status word of `ws` when device_status is
 * NULL, and leave the affected entries empty (unchanged when the page of the last token itself
 * is missing).  `ws` is the workspace of the attention call that will read the arrays: its next
 * launch is then issued without programmatic dependent launch, because the attention prologue
 * reads the lists ahead of the dependency wait.  With ws == NULL that ordering is the caller's
 * job: put another kernel between this call and the attention call, or switch programmatic
 * dependent launch off (kap_set_launch_options).
 * Errors: KAP_ERR_UNSUPPORTED (page_size > 16), KAP_ERR_INVALID_ARG, KAP_ERR_CUDA.
 */
kap_status kap_compile_growing_plan(
    int32_t batch, int32_t page_size,
    const int32_t* ctx_len, const int32_t* span_indptr, const int32_t* span_start,
    const int32_t* span_len, const float* span_score, const int32_t* budget_tokens,
    const int32_t* n_sink, const int32_t* n_recent, const uint8_t* force_full, float s_max,
    const int32_t* bt_indptr, const int32_t* bt_pages,   /* HOST, as kap_compile_plan; required */
    int32_t max_growth,                /* tokens a full-context sequence may still grow by */
    int64_t plan_capacity,
    int32_t* plan_indptr,              /* HOST out [batch+1], reserved entries included */
    int32_t* plan_logical_pages,       /* HOST out */
    int32_t* plan_phys_pages,          /* HOST out */
    uint16_t* plan_token_masks,        /* HOST out */
    int32_t* plan_flags,               /* HOST out [batch] */
    int32_t* selected_tokens,          /* HOST out [batch] or NULL */
    int32_t* tail_desc);               /* HOST out [batch][3] */

kap_status kap_refresh_recent(
    const int32_t* plan_indptr,        /* DEVICE [batch+1] */
    int32_t* plan_logical_pages,       /* DEVICE in/out */
    int32_t* plan_phys_pages,          /* DEVICE in/out */
    uint16_t* plan_token_masks,        /* DEVICE in/out */
    const int32_t* tail_desc,          /* DEVICE [batch][3] */
    const int32_t* bt_indptr,          /* DEVICE [batch+1] */
    const int32_t* bt_pages,           /* DEVICE */
    const int32_t* ctx_len,            /* DEVICE [batch] current lengths */
    int32_t batch, int32_t page_size, int64_t num_pool_pages,
    int32_t* device_status,            /* DEVICE or NULL */
    kap_workspace* ws,                 /* or NULL */
    void* cuda_stream);

/*
 * kap_materialize_view - the paper's selected-KV view as a physical copy (Section 3.1,
 * "Selected-KV view materialization": the plan's pages are laid out compactly in a reusable
 * workspace and a compact block table maps the plan's logical blocks to the compact pages).
 * compact_pool[i] = kv_pool[plan_phys_pages[i]] for i < n_selected, compact_pages[i] = i; logical
 * page indices are untouched (positions are preserved).  kap_selected_decode_attn run on
 * (compact_pool, compact_pages, plan_logical_pages) then equals the in-place call bit for bit.
 * This library's attention gathers in place and does not need the copy; the call is here for
 * comparison and for back ends that want a dense view.
 * Pages are copied whole, so the call serves either pool layout.  Token masks and logical pages
 * are indexed by list position and apply to the copy unchanged.
 * n_selected > compact_capacity is the paper's "plan exceeds the workspace" fallback condition:
 * KAP_ERR_CAPACITY, nothing enqueued.  A source page outside the pool is reported in
 * *device_status (1 << KAP_ERR_DEVICE_INDEX) and not copied.  Other errors: KAP_ERR_UNSUPPORTED
 * (shape), KAP_ERR_INVALID_ARG, KAP_ERR_CUDA.  Asynchronous on cuda_stream.
 */
kap_status kap_materialize_view(
    const void* kv_pool, int64_t num_pool_pages,   /* DEVICE bf16 [pages][2][Hkv][P][d] */
    const int32_t* plan_phys_pages,                /* DEVICE [n_selected] */
    int64_t n_selected,
    int32_t num_kv_heads, int32_t head_dim, int32_t page_size,
    void* compact_pool, int64_t compact_capacity,  /* DEVICE bf16 [capacity][2][Hkv][P][d] */
    int32_t* compact_pages,                        /* DEVICE out [n_selected] or NULL */
    int32_t* device_status,                        /* DEVICE int32 or NULL */
    void* cuda_stream);

/*
 * kap_selected_decode_attn_static - the proposal-path attention of kap_selected_decode_attn for
 * callers that are not allowed to allocate device memory.  (The paper has no counterpart: this is
 * a packaging of the same computation, not another operation.)
 *
 * Who needs it: code that runs inside a host program which reserved the whole GPU up front and
 * hands out memory through its own pool (an inference server, a plug-in loaded into one), code on
 * a path where cudaMalloc's implicit device synchronisation is not acceptable, or code that simply
 * has no safe point at which to create and later destroy a kap_workspace.  Such callers cannot use
 * the workspace entry points, because kap_workspace_create allocates.
 *
 * What is different from kap_selected_decode_attn:
 *   - no kap_workspace and no kap_schedule.  Every (sequence, KV head) page list is cut into
 *     `num_splits` near-equal slices by a small kernel on the device; the work list, the merge map,
 *     the fp32 partial results and the status word live in one array built into the library
 *     (4 MiB of device memory on every GPU that loads it, held until the process exits).
 *   - the call makes no cudaMalloc / cudaFree and calls no allocating library routine.  The first
 *     call on a device looks up the array's device address and sets a kernel attribute (once per
 *     device, for the device that is current at that moment); make that first call outside any
 *     stream capture.
 *   - sizes the array cannot hold are refused: batch * num_kv_heads * num_splits work items need
 *     about 32 + (Hq/Hkv) * 520 bytes each; beyond 4 MiB in total the call returns
 *     KAP_ERR_CAPACITY and enqueues nothing (with 32/8 heads: roughly 1900 work items).
 *   - one slice (ceil(list pages / num_splits) pages of one sequence) is run by one CTA, which can
 *     hold 640 page ids, or 1600 when plan_logical_pages is NULL.  The list lengths are on the
 *     device, so the host cannot refuse a longer slice up front: the device cuts it to the limit,
 *     sets 1 << KAP_ERR_CAPACITY in the status word and the output of that sequence is NOT valid
 *     (the pages beyond the cut were not attended to).  A caller that passes device_status == NULL
 *     gets no signal at all, so choose num_splits >= ceil(longest list / 640) (or / 1600): a
 *     full-context list of 131 072 tokens (8192 pages) needs 13 splits with logical indices,
 *     6 without.
 *   - all calls on a device share the array and it keeps the previous call's contents.  The call
 *     itself clears the only part that must start at zero (the status word) and rewrites the
 *     rest before use, so back-to-back calls on ONE stream are fine; calls that may overlap on
 *     the GPU (different streams, different host threads) race on the array and must be ordered
 *     by the caller.
 *   - kernels are launched without programmatic stream serialisation (the work list is produced
 *     on the device just before it is read).
 *   - page-granular visibility and the head-major (KAP_KV_HND) pool layout only: token masks and
 *     the token-major layout belong to the workspace entry point.
 * Results are the same as the workspace entry point's up to the order of the fp32 sums.
 * device_status (DEVICE int32, may be NULL) receives the kernels' status bits after the call's
 * kernels: 0, or a bit-or of 1 << KAP_ERR_DEVICE_INDEX (a page id outside the pool), 1 <<
 * KAP_ERR_TIMEOUT and 1 << KAP_ERR_CAPACITY (a slice was cut, see above).
 * Errors: KAP_ERR_UNSUPPORTED (shape), KAP_ERR_INVALID_ARG (NULL pointer, num_splits < 1,
 * misaligned pool), KAP_ERR_CAPACITY (scratch size, or batch > 16 383), KAP_ERR_CUDA.
 */
kap_status kap_selected_decode_attn_static(
    const void* q,                     /* DEVICE bf16 [batch, Hq, d] */
    const void* kv_pool,               /* DEVICE bf16 [num_pool_pages][2][Hkv][P][d] */
    int64_t num_pool_pages,
    const int32_t* plan_indptr,        /* DEVICE [batch+1] */
    const int32_t* plan_phys_pages,    /* DEVICE */
    const int32_t* plan_logical_pages, /* DEVICE or NULL */
    const int32_t* ctx_len,            /* DEVICE [batch] */
    int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t page_size,
    float sm_scale,
    int32_t num_splits,                /* slices per (sequence, KV head), >= 1 */
    void* out,                         /* DEVICE bf16 [batch, Hq, d] */
    float* lse,                        /* DEVICE fp32 [batch, Hq] or NULL */
    int32_t* device_status,            /* DEVICE int32 or NULL */
    void* cuda_stream);

/*
 * kap_device_sm_rates - relative memory-streaming rate of every SM of a device (mean 1.0), measured
 * once per process on first use (about a millisecond; allocates and frees a temporary buffer of
 * 3 MiB per SM).  On B200 groups of 8 to 10 SMs share a fixed-bandwidth port towards L2 / HBM, so
 * while all SMs stream an SM of a larger group is served up to 20 % slower; kap_schedule uses these
 * rates to size the slices of full-context launches.  The paper has no counterpart.
 * rates may be NULL (then only *n_sms is written).  Errors: KAP_ERR_CUDA, KAP_ERR_CAPACITY.
 */
kap_status kap_device_sm_rates(int32_t device, int32_t capacity, float* rates /* HOST out */, int32_t* n_sms);

/* Synchronises `cuda_stream` and returns the device status word of the workspace (KAP_OK,
 * KAP_ERR_TIMEOUT or KAP_ERR_DEVICE_INDEX), clearing it. */
kap_status kap_workspace_check(kap_workspace* ws, void* cuda_stream);

/* Tuning knobs of the attention launches, process-wide; a negative value keeps the setting.
 *   use_pdl      != 0 (default): launch with programmatic stream serialisation, so that a kernel's
 *                prologue overlaps the tail of the previous kernel on the stream when that kernel
 *                releases its dependents early (this library's kernels do; ordinary kernels
 *                release them only when they complete, which changes nothing).  Before the
 *                previous kernel has completed an attention kernel reads only static metadata:
 *                the work list, the page lists and q_indptr.  Those arrays must therefore be
 *                final before the previous kernel was launched.
 *   early_kv     != 0 (default; needs use_pdl): in that window the kernel also reads ctx_len as a
 *                hint and starts loading KV pages that hold only tokens older than the query
 *                rows' own (t < ctx_len - n_q) - pages written in earlier decoding steps.  Those
 *                pages must then be final under the same rule; ctx_len may be advanced by the
 *                kernels still running by at most n_q, or lowered (the masks use the value read
 *                after the wait); Q, the pages holding the rows' own tokens, out and lse may still
 *                be written by them.  kap_append_kv with several new tokens per sequence
 *                (new_indptr given) could break the first condition for the attention call that
 *                follows it ON THE SAME STREAM, so the library starts that one launch's loads after
 *                the wait; the bookkeeping is per stream, attention calls on other streams neither
 *                lose their early loads nor use the mark up.
 *   ctas_per_sm  resident CTAs per SM the scheduler fills in one wave; 0 = as many as fit.
 *   max_cluster  largest thread-block cluster (1 .. 16; default 16, sizes above 8 use the
 *                non-portable cluster launch) the scheduler may give a work item.  The CTAs of a cluster share the item's pages and reduce their partial
 *                results through distributed shared memory, so a (sequence, KV head) that fits one
 *                cluster needs no merge pass.
 *   ring_slots   page slots (8 KiB each) in a CTA's shared-memory ring: 8 (3 CTAs per SM), 12 or 16
 *                (2 per SM) or 24 (1 per SM); more slots = more loads in flight per CTA.
 * ctas_per_sm, max_cluster and ring_slots take effect at the next kap_schedule.  The paper has no
 * counterpart for these.  Error: KAP_ERR_INVALID_ARG for a max_cluster outside 1 .. 16 or
 * a ring_slots that is not 8, 12, 16 or 24. */
kap_status kap_set_launch_options(int32_t use_pdl, int32_t early_kv, int32_t ctas_per_sm,
                                  int32_t max_cluster, int32_t ring_slots);

/* Which kernel runs kap_verify_attn (Section 3.2 "Full-context verification"); takes effect at the
 * next kap_schedule of a verification workspace, process-wide.
 *   0 (default)  the split kernel: mma.sync tiles of 16 query rows per warp.
 *   1            the tcgen05 kernel: one tcgen05.mma per four pages for all query rows of a KV head,
 *                accumulators in tensor memory, at most 32 query rows per KV head (n_q * Hq / Hkv;
 *                schedules with more rows use the split kernel), slices of at most 1024 pages per
 *                CTA, a 12-slot ring and two CTAs per SM whatever kap_set_launch_options says, no
 *                clusters.  Same results within the tolerance of the path; on the paper-shaped
 *                workloads it is the slower of the two on B200 by 10-20 % (it keeps a page longer
 *                in its ring slot), which is why it is not the default.
 * The paper has no counterpart.  Error: KAP_ERR_INVALID_ARG for any other value. */
kap_status kap_set_verify_kernel(int32_t kernel);

/* Number of kernels this library has launched in this process (all threads). */
int64_t kap_launch_count(void);

/* Thread-local text for the last non-OK status returned on this thread ("" if none). */
const char* kap_last_error(void);

/* "kap-b200 <major>.<minor> sm_100a" */
const char* kap_version(void);

#ifdef __cplusplus
}
#endif
#endif /* KAP_H_ */
