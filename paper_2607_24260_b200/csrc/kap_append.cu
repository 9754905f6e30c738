// kap_append_kv: place newly scheduled tokens' K/V rows into their physical KV slots through the
// block table (the slot mapping of the KAP paper, Section 3.1 "Selected-KV view materialization";
// every proposal step and the verifier pass write the K/V of the tokens they process, Section 3.2).
// One CTA per sequence, so the optional ctx_len update cannot race with another CTA's reads.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <atomic>

#include "kap_internal.h"

namespace kap {
void count_launch();
void kv_written_in_bulk(void* cuda_stream);

namespace {

__global__ void __launch_bounds__(256)
kap_append_kv_kernel(const uint4* __restrict__ k_new, const uint4* __restrict__ v_new,
                     const int32_t* __restrict__ new_indptr, uint4* __restrict__ pool,
                     long long num_pool_pages, const int32_t* __restrict__ bt_indptr,
                     const int32_t* __restrict__ bt_pages, int32_t* ctx_len, int advance, int hkv,
                     int nhd, int32_t* status)
{
    constexpr int kRowVec = kHeadDim * 2 / 16;                 // 16 uint4 per 128-element bf16 row
    const int b = blockIdx.x;
    const int row0 = new_indptr ? new_indptr[b] : b;
    const int n_new = new_indptr ? new_indptr[b + 1] - row0 : 1;
    const int L = ctx_len[b];
    const int n_bt = bt_indptr[b + 1] - bt_indptr[b];
    const long long page_vec = 2ll * hkv * kPageSize * kRowVec;   // uint4 per page
    // one (token, K|V, head, 16-byte piece) per thread iteration
    const int total = n_new * 2 * hkv * kRowVec;
    for (int i = threadIdx.x; i < total; i += blockDim.x) {
        const int piece = i % kRowVec;
        const int g = (i / kRowVec) % hkv;
        const int kv = (i / (kRowVec * hkv)) & 1;
        const int j = i / (kRowVec * hkv * 2);
        const long long pos = (long long)L + j;
        const long long lp = pos / kPageSize;
        int32_t page = lp < n_bt ? bt_pages[bt_indptr[b] + lp] : -1;
        if (L < 0 || page < 0 || page >= num_pool_pages) {       // report, never write out of range
            if (status) atomicOr(status, 1 << KAP_ERR_DEVICE_INDEX);
            continue;
        }
        const uint4* src = (kv ? v_new : k_new) + ((long long)(row0 + j) * hkv + g) * kRowVec + piece;
        // row of (K|V, head g, slot) inside the page: head-major ("HND") or token-major ("NHD")
        const long long row = nhd ? ((long long)kv * kPageSize + pos % kPageSize) * hkv + g
                                  : (long long)(kv * hkv + g) * kPageSize + pos % kPageSize;
        pool[page * page_vec + row * kRowVec + piece] = *src;
    }
    if (advance) {
        __syncthreads();                                         // every thread has read L
        if (threadIdx.x == 0) ctx_len[b] = L + n_new;
    }
}

}  // namespace
}  // namespace kap

extern "C" kap_status kap_append_kv(
    const void* k_new, const void* v_new, const int32_t* new_indptr, void* kv_pool,
    int64_t num_pool_pages, const int32_t* bt_indptr, const int32_t* bt_pages, int32_t* ctx_len,
    int32_t advance, int32_t batch, int32_t num_kv_heads, int32_t head_dim, int32_t page_size,
    int32_t kv_layout, int32_t* device_status, void* cuda_stream)
{
    using namespace kap;
    if (head_dim != kHeadDim || page_size != kPageSize)
        return fail(KAP_ERR_UNSUPPORTED, "head_dim %d / page_size %d (supported: 128 / 16)", head_dim, page_size);
    if (batch < 0 || num_kv_heads <= 0) return fail(KAP_ERR_INVALID_ARG, "batch %d / num_kv_heads %d", batch, num_kv_heads);
    if (kv_layout != KAP_KV_HND && kv_layout != KAP_KV_NHD)
        return fail(KAP_ERR_INVALID_ARG, "kv_layout %d (KAP_KV_HND = 0, KAP_KV_NHD = 1)", kv_layout);
    if (batch == 0) return KAP_OK;
    if (!k_new || !v_new || !kv_pool || !bt_indptr || !bt_pages || !ctx_len || num_pool_pages <= 0)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer or empty pool");
    if ((reinterpret_cast<uintptr_t>(k_new) | reinterpret_cast<uintptr_t>(v_new) |
         reinterpret_cast<uintptr_t>(kv_pool)) & 15)
        return fail(KAP_ERR_INVALID_ARG, "k_new, v_new and kv_pool must be 16-byte aligned");
    kap_append_kv_kernel<<<(unsigned)batch, 256, 0, (cudaStream_t)cuda_stream>>>(
        (const uint4*)k_new, (const uint4*)v_new, new_indptr, (uint4*)kv_pool, num_pool_pages, bt_indptr,
        bt_pages, ctx_len, advance, num_kv_heads, kv_layout == KAP_KV_NHD, device_status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return fail(KAP_ERR_CUDA, "kap_append_kv launch failed: %s", cudaGetErrorString(e));
    count_launch();
    // with several new tokens per sequence the early page loads of the next attention kernel on
    // this stream could touch tokens this kernel is still writing: that launch starts its loads
    // after the dependency wait
    if (new_indptr) kv_written_in_bulk(cuda_stream);
    return KAP_OK;
}
