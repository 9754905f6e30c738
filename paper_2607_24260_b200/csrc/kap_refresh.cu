// kap_refresh_recent: keep a compiled plan valid while the context grows, without recompiling it.
// A growing plan (kap_compile_growing_plan) lists the pages of the tokens that stay selected at
// every length - the attention-sink prefix and the selected evidence spans (Algorithm 1, Section
// 3.1), or the whole prefix for a full-context plan - followed by a few reserved entries per
// sequence.  This kernel rewrites the reserved entries from the current device-side ctx_len: the
// pages of the recent window [L - n_recent, L) (Section 3.2: each proposal step sees the tokens
// written before it), with a 16-bit token mask that leaves out the tokens the fixed part already
// holds, so that no token is counted twice.  Unused reserved entries repeat the sequence's last
// page with an empty mask: the attention kernel reads it like any page and it contributes nothing.
#include <cuda_runtime.h>

#include "kap_internal.h"

namespace kap {
void count_launch();
int32_t* workspace_status_word(kap_workspace* ws);
void workspace_lists_rewritten(kap_workspace* ws);

namespace {

__global__ void __launch_bounds__(32)
kap_refresh_recent_kernel(const int32_t* __restrict__ plan_indptr, int32_t* plan_logical,
                          int32_t* plan_phys, uint16_t* plan_masks,
                          const int32_t* __restrict__ tail_desc, const int32_t* __restrict__ bt_indptr,
                          const int32_t* __restrict__ bt_pages, const int32_t* __restrict__ ctx_len,
                          int page_size, long long num_pool_pages, int32_t* status)
{
    const int b = blockIdx.x;
    const int reserved = tail_desc[b * 3 + 0];
    const long long window = tail_desc[b * 3 + 1];
    const long long from = tail_desc[b * 3 + 2];
    const long long L = ctx_len[b];
    const int list_end = plan_indptr[b + 1];
    const int tail0 = list_end - reserved;                 // the fixed part is [list0, tail0)
    const int list0 = plan_indptr[b];
    if (reserved < 0 || tail0 < list0 || L <= 0) {
        if (threadIdx.x == 0 && status) atomicOr(status, 1 << KAP_ERR_DEVICE_INDEX);
        return;
    }
    long long lo = L - window;                             // first token of the moving part
    if (lo < from) lo = from;
    if (lo < 0) lo = 0;
    const long long first_page = lo / page_size;
    const long long needed = L > lo ? (L - 1) / page_size - first_page + 1 : 0;
    if (needed > reserved && threadIdx.x == 0 && status)   // the context outgrew the reservation
        atomicOr(status, 1 << KAP_ERR_DEVICE_INDEX);
    const int n_bt = bt_indptr[b + 1] - bt_indptr[b];
    // an entry that lists nothing still names a page the kernel will read: the last page of the
    // context (its rows below the length hold real tokens, the kernel zeroes the rest)
    const long long last_page = (L - 1) / page_size;
    const int32_t idle_phys = last_page < n_bt ? bt_pages[bt_indptr[b] + last_page] : -1;
    if (idle_phys < 0 || idle_phys >= num_pool_pages) {
        if (threadIdx.x == 0 && status) atomicOr(status, 1 << KAP_ERR_DEVICE_INDEX);
        return;                                            // entries keep their previous contents
    }
    for (int r = threadIdx.x; r < reserved; r += blockDim.x) {
        int32_t logical = (int32_t)last_page, phys = idle_phys;
        uint32_t bits = 0;
        if (r < needed) {
            const long long p = first_page + r;
            const long long t0 = max(lo, p * page_size) - p * page_size;
            const long long t1 = min(L, (p + 1) * page_size) - p * page_size;
            bits = ((1u << t1) - 1u) & ~((1u << t0) - 1u);
            // tokens of this page that the fixed part already lists (ascending pages: bisect)
            int a = list0, z = tail0;
            while (a < z) {
                const int mid = (a + z) >> 1;
                if (plan_logical[mid] < p) a = mid + 1; else z = mid;
            }
            if (a < tail0 && plan_logical[a] == p) bits &= ~(uint32_t)plan_masks[a];
            const int32_t page = p < n_bt ? bt_pages[bt_indptr[b] + p] : -1;
            if (page < 0 || page >= num_pool_pages) {
                if (status) atomicOr(status, 1 << KAP_ERR_DEVICE_INDEX);
                bits = 0;
            } else {
                logical = (int32_t)p;
                phys = page;
            }
        }
        plan_logical[tail0 + r] = logical;
        plan_phys[tail0 + r] = phys;
        plan_masks[tail0 + r] = (uint16_t)bits;
    }
}

}  // namespace
}  // namespace kap

extern "C" kap_status kap_refresh_recent(
    const int32_t* plan_indptr, int32_t* plan_logical_pages, int32_t* plan_phys_pages,
    uint16_t* plan_token_masks, const int32_t* tail_desc, const int32_t* bt_indptr,
    const int32_t* bt_pages, const int32_t* ctx_len, int32_t batch, int32_t page_size,
    int64_t num_pool_pages, int32_t* device_status, kap_workspace* ws, void* cuda_stream)
{
    using namespace kap;
    if (page_size <= 0 || page_size > 16)
        return fail(KAP_ERR_UNSUPPORTED, "page_size %d (token masks hold 16 bits)", page_size);
    if (batch < 0) return fail(KAP_ERR_INVALID_ARG, "batch %d < 0", batch);
    if (batch == 0) return KAP_OK;
    if (!plan_indptr || !plan_logical_pages || !plan_phys_pages || !plan_token_masks || !tail_desc ||
        !bt_indptr || !bt_pages || !ctx_len || num_pool_pages <= 0)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer or empty pool");
    int32_t* status = device_status ? device_status : (ws ? workspace_status_word(ws) : nullptr);
    kap_refresh_recent_kernel<<<(unsigned)batch, 32, 0, (cudaStream_t)cuda_stream>>>(
        plan_indptr, plan_logical_pages, plan_phys_pages, plan_token_masks, tail_desc, bt_indptr,
        bt_pages, ctx_len, page_size, num_pool_pages, status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(KAP_ERR_CUDA, "kap_refresh_recent launch failed: %s", cudaGetErrorString(e));
    count_launch();
    // the attention kernels read the lists in their prologue, ahead of the stream dependency when
    // launched programmatically: the next launch on this workspace must be an ordinary one
    if (ws) workspace_lists_rewritten(ws);
    return KAP_OK;
}
