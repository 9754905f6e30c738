// kap_materialize_view: the paper's selected-KV view as a physical copy (Section 3.1, "Selected-KV
// view materialization": the selected pages are compacted into a reusable workspace and a compact
// block table resolves the plan's logical blocks to compact pages).  This library's attention
// gathers the plan's pages in place and does not need the copy; the call exists so that the two
// designs can be compared and for back ends that want a dense view.
#include <cuda_runtime.h>

#include "kap_internal.h"

namespace kap {
void count_launch();

namespace {

constexpr int kSlicesPerPage = 4;

__global__ void __launch_bounds__(256)
kap_copy_pages_kernel(const uint4* __restrict__ pool, long long num_pool_pages,
                      const int32_t* __restrict__ phys_pages, uint4* __restrict__ compact,
                      int32_t* __restrict__ compact_pages, long long page_vec, int32_t* status)
{
    const long long i = blockIdx.x;
    const int32_t src_page = phys_pages[i];
    if (blockIdx.y == 0 && threadIdx.x == 0 && compact_pages) compact_pages[i] = (int32_t)i;
    if (src_page < 0 || src_page >= num_pool_pages) {          // report, copy nothing
        if (threadIdx.x == 0 && status) atomicOr(status, 1 << KAP_ERR_DEVICE_INDEX);
        return;
    }
    const long long slice = page_vec / kSlicesPerPage;
    const uint4* src = pool + src_page * page_vec + blockIdx.y * slice;
    uint4* dst = compact + i * page_vec + blockIdx.y * slice;
    for (long long v = threadIdx.x; v < slice; v += 4 * blockDim.x) {
        uint4 x[4];
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (v + u * blockDim.x < slice) x[u] = __ldcs(src + v + u * blockDim.x);
#pragma unroll
        for (int u = 0; u < 4; ++u)
            if (v + u * blockDim.x < slice) dst[v + u * blockDim.x] = x[u];
    }
}

}  // namespace
}  // namespace kap

extern "C" kap_status kap_materialize_view(
    const void* kv_pool, int64_t num_pool_pages, const int32_t* plan_phys_pages, int64_t n_selected,
    int32_t num_kv_heads, int32_t head_dim, int32_t page_size, void* compact_pool,
    int64_t compact_capacity, int32_t* compact_pages, int32_t* device_status, void* cuda_stream)
{
    using namespace kap;
    if (head_dim != kHeadDim || page_size != kPageSize)
        return fail(KAP_ERR_UNSUPPORTED, "head_dim %d / page_size %d (supported: 128 / 16)", head_dim, page_size);
    if (n_selected < 0 || num_kv_heads <= 0 || num_pool_pages <= 0 || compact_capacity < 0)
        return fail(KAP_ERR_INVALID_ARG, "negative size");
    if (n_selected > compact_capacity)
        return fail(KAP_ERR_CAPACITY, "the plan selects %lld pages, the compact workspace holds %lld "
                    "(the paper's fallback condition: use full-context access)", (long long)n_selected,
                    (long long)compact_capacity);
    if (n_selected == 0) return KAP_OK;
    if (!kv_pool || !plan_phys_pages || !compact_pool)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer");
    if ((reinterpret_cast<uintptr_t>(kv_pool) | reinterpret_cast<uintptr_t>(compact_pool)) & 15)
        return fail(KAP_ERR_INVALID_ARG, "pools must be 16-byte aligned");
    if (n_selected > 0x7fffffffLL) return fail(KAP_ERR_UNSUPPORTED, "more than 2^31 pages");
    const long long page_vec = 2ll * num_kv_heads * kPageSize * kHeadDim * 2 / 16;    // uint4 per page
    if (page_vec % kSlicesPerPage) return fail(KAP_ERR_UNSUPPORTED, "num_kv_heads %d", num_kv_heads);
    kap_copy_pages_kernel<<<dim3((unsigned)n_selected, kSlicesPerPage), 256, 0, (cudaStream_t)cuda_stream>>>(
        (const uint4*)kv_pool, num_pool_pages, plan_phys_pages, (uint4*)compact_pool, compact_pages, page_vec,
        device_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(KAP_ERR_CUDA, "kap_materialize_view launch failed: %s", cudaGetErrorString(e));
    count_launch();
    return KAP_OK;
}
