// kap_top3_accept: the verifier's acceptance rule of the KAP paper (Section 3.2, Eq. 2 and the
// Top-3 instantiation of the verification policy): a proposed token is accepted when it is among
// the target model's three highest-scoring candidates at its position; m = length of the accepted
// prefix; the next carry token is the verifier's own best candidate at the first position that
// was not accepted (the bonus position when everything was accepted).
//
// Kernel 1: one CTA per logits row finds the row's top 3 (value descending, index ascending on
// ties, NaN ranked below everything) - a pure streaming reduction over the vocabulary.
// Kernel 2: one thread per sequence walks its rows.
#include <cuda_runtime.h>

#include <cfloat>

#include "kap_internal.h"

namespace kap {
void count_launch();

namespace {

struct Top3 { float v[3]; int i[3]; };

// strict "a ranks before b": higher value first, then lower index
__device__ __forceinline__ bool before(float va, int ia, float vb, int ib) {
    return va > vb || (va == vb && ia < ib);
}
__device__ __forceinline__ void push(Top3& t, float v, int i) {
    if (!(v == v)) v = -INFINITY;                                  // NaN ranks last
    if (!before(v, i, t.v[2], t.i[2])) return;
    if (before(v, i, t.v[0], t.i[0])) {
        t.v[2] = t.v[1]; t.i[2] = t.i[1]; t.v[1] = t.v[0]; t.i[1] = t.i[0]; t.v[0] = v; t.i[0] = i;
    } else if (before(v, i, t.v[1], t.i[1])) {
        t.v[2] = t.v[1]; t.i[2] = t.i[1]; t.v[1] = v; t.i[1] = i;
    } else {
        t.v[2] = v; t.i[2] = i;
    }
}
__device__ __forceinline__ Top3 empty_top3() {
    Top3 t;
#pragma unroll
    for (int k = 0; k < 3; ++k) { t.v[k] = -INFINITY; t.i[k] = INT32_MAX; }
    return t;
}

__global__ void __launch_bounds__(256)
kap_top3_rows_kernel(const float* __restrict__ logits, long long row_stride, int vocab,
                     int32_t* __restrict__ top3)
{
    const float* row = logits + (long long)blockIdx.x * row_stride;
    Top3 t = empty_top3();
    // 16-byte loads where the row allows it, scalar head and tail otherwise
    const int head = min(vocab, (int)(((16 - (reinterpret_cast<uintptr_t>(row) & 15)) & 15) / 4));
    for (int i = threadIdx.x; i < head; i += blockDim.x) push(t, row[i], i);
    const int n4 = (vocab - head) / 4;
    const float4* row4 = reinterpret_cast<const float4*>(row + head);
    for (int j = threadIdx.x; j < n4; j += blockDim.x) {
        const float4 x = __ldcs(row4 + j);
        const int i = head + 4 * j;
        push(t, x.x, i); push(t, x.y, i + 1); push(t, x.z, i + 2); push(t, x.w, i + 3);
    }
    for (int i = head + 4 * n4 + threadIdx.x; i < vocab; i += blockDim.x) push(t, row[i], i);
    // warp merge, then the 8 warps through shared memory
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Top3 o;
#pragma unroll
        for (int k = 0; k < 3; ++k) {
            o.v[k] = __shfl_xor_sync(0xffffffffu, t.v[k], off);
            o.i[k] = __shfl_xor_sync(0xffffffffu, t.i[k], off);
        }
#pragma unroll
        for (int k = 0; k < 3; ++k) push(t, o.v[k], o.i[k]);
    }
    __shared__ Top3 part[8];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
#pragma unroll
            for (int k = 0; k < 3; ++k) push(t, part[w].v[k], part[w].i[k]);
#pragma unroll
        for (int k = 0; k < 3; ++k) top3[(long long)blockIdx.x * 3 + k] = t.i[k];
    }
}

__global__ void kap_accept_prefix_kernel(const int32_t* __restrict__ top3, const int32_t* __restrict__ row_indptr,
                                         const int32_t* __restrict__ proposed, int batch,
                                         int32_t* __restrict__ accepted, int32_t* __restrict__ next_token)
{
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= batch) return;
    const int r0 = row_indptr[b], n = row_indptr[b + 1] - r0;     // n = k + 1 rows
    int m = 0;
    if (n <= 0) { accepted[b] = 0; next_token[b] = -1; return; }
    while (m < n - 1) {
        const int tok = proposed[r0 + m];
        const int32_t* c = top3 + (long long)(r0 + m) * 3;
        if (tok != c[0] && tok != c[1] && tok != c[2]) break;
        ++m;
    }
    accepted[b] = m;
    next_token[b] = top3[(long long)(r0 + m) * 3];
}

}  // namespace
}  // namespace kap

extern "C" kap_status kap_top3_accept(
    const float* logits, int64_t row_stride, const int32_t* row_indptr, const int32_t* proposed,
    int32_t batch, int32_t total_rows, int32_t vocab, int32_t* top3, int32_t* accepted,
    int32_t* next_token, void* cuda_stream)
{
    using namespace kap;
    if (batch < 0 || total_rows < 0 || vocab < 3 || row_stride < vocab)
        return fail(KAP_ERR_INVALID_ARG, "batch %d, rows %d, vocab %d, row_stride %lld", batch, total_rows,
                    vocab, (long long)row_stride);
    if (batch == 0 || total_rows == 0) return KAP_OK;
    if (!logits || !row_indptr || !proposed || !top3 || !accepted || !next_token)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer");
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    kap_top3_rows_kernel<<<(unsigned)total_rows, 256, 0, stream>>>(logits, row_stride, vocab, top3);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess) {
        count_launch();
        kap_accept_prefix_kernel<<<(unsigned)((batch + 127) / 128), 128, 0, stream>>>(top3, row_indptr, proposed,
                                                                                    batch, accepted, next_token);
        e = cudaGetLastError();
        if (e == cudaSuccess) count_launch();
    }
    if (e != cudaSuccess) return fail(KAP_ERR_CUDA, "kap_top3_accept launch failed: %s", cudaGetErrorString(e));
    return KAP_OK;
}
