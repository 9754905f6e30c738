// kap_top3_accept: the verifier's acceptance rule of the KAP paper (Section 3.2, Eq. 2 and the
// Top-3 instantiation of the verification policy): a proposed token is accepted when it is among
// the target model's three highest-scoring candidates at its position; m = length of the accepted
// prefix; the next carry token is the verifier's own best candidate at the first position that
// was not accepted (the bonus position when everything was accepted).
//
// Kernel 1: a cluster of up to 8 CTAs per logits row finds the row's top 3 (value descending, index ascending on
// ties, NaN ranked below everything, -inf included) - a pure streaming reduction over the vocabulary.
// Kernel 2: one thread per sequence walks its rows.
#include <cuda_runtime.h>

#include <cfloat>
#include <mutex>

#include "kap_internal.h"

namespace kap {
void count_launch();

namespace {

// A candidate is one 64-bit key that sorts the way the rule ranks: the logit mapped to an
// order-preserving unsigned integer in the high word (NaN -> 0, below -inf), the complemented index
// in the low word (lower index wins ties).  Keeping the best three is then five branch-free
// max / min operations per logit - no divergence, whatever the data.
typedef unsigned long long Key;
struct Top3 { Key k[3]; };                                     // k[0] >= k[1] >= k[2]; 0 = empty

__device__ __forceinline__ Key make_key(float v, int i) {
    uint32_t u = __float_as_uint(v + 0.0f);                     // -0.0 and +0.0 are the same value
    u = (v != v) ? 0u : (u ^ ((u >> 31) ? 0xffffffffu : 0x80000000u));
    return ((Key)u << 32) | (uint32_t)~i;
}
__device__ __forceinline__ int key_index(Key k) { return (int)~(uint32_t)k; }
__device__ __forceinline__ void push(Top3& t, Key x) {
    const Key b0 = max(t.k[0], x), r1 = min(t.k[0], x);
    const Key b1 = max(t.k[1], r1), r2 = min(t.k[1], r1);
    t.k[0] = b0; t.k[1] = b1; t.k[2] = max(t.k[2], r2);
}
__device__ __forceinline__ Top3 empty_top3() { Top3 t; t.k[0] = t.k[1] = t.k[2] = 0; return t; }

// grid = rows * S CTAs in clusters of S: the S CTAs of a cluster share one row (a slice of the
// vocabulary each) and the cluster's first CTA merges their candidates through distributed
// shared memory.
__global__ void __launch_bounds__(256)
kap_top3_rows_kernel(const float* __restrict__ logits, long long row_stride, int vocab, int S,
                     int32_t* __restrict__ top3)
{
    const int r = blockIdx.x / S, part_id = blockIdx.x % S;
    const float* row = logits + (long long)r * row_stride;
    const int per = (vocab + S - 1) / S;
    const int lo = min(vocab, part_id * per), hi = min(vocab, lo + per);
    Top3 t = empty_top3();
    // 16-byte loads where the slice allows it, scalar head and tail otherwise
    const int head = min(hi - lo, (int)(((16 - (reinterpret_cast<uintptr_t>(row + lo) & 15)) & 15) / 4));
    for (int i = lo + threadIdx.x; i < lo + head; i += blockDim.x) push(t, make_key(row[i], i));
    const int n4 = (hi - lo - head) / 4;
    const float4* row4 = reinterpret_cast<const float4*>(row + lo + head);
    for (int j0 = threadIdx.x; j0 < n4; j0 += 8 * blockDim.x) {       // eight loads in flight per thread
        float4 x[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int j = j0 + u * blockDim.x;
            if (j < n4) x[u] = __ldcs(row4 + j);
        }
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int j = j0 + u * blockDim.x;
            if (j < n4) {
                const int i = lo + head + 4 * j;
                push(t, make_key(x[u].x, i)); push(t, make_key(x[u].y, i + 1));
                push(t, make_key(x[u].z, i + 2)); push(t, make_key(x[u].w, i + 3));
            }
        }
    }
    for (int i = lo + head + 4 * n4 + threadIdx.x; i < hi; i += blockDim.x) push(t, make_key(row[i], i));
    // warp merge, then the 8 warps through shared memory
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) {
        Key o[3];
#pragma unroll
        for (int k = 0; k < 3; ++k) o[k] = __shfl_xor_sync(0xffffffffu, t.k[k], off);
#pragma unroll
        for (int k = 0; k < 3; ++k) push(t, o[k]);
    }
    __shared__ Top3 part[8];
    __shared__ Top3 cta_best;
    __shared__ Top3 peers[8];
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = t;
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
#pragma unroll
            for (int k = 0; k < 3; ++k) push(t, part[w].k[k]);
        cta_best = t;
    }
    if (S > 1) {
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
        // thread p of the first CTA fetches peer p's candidates (all peers in parallel), thread 0
        // merges them
        if (part_id == 0 && threadIdx.x >= 1 && threadIdx.x < S) {
            uint32_t addr;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
                         : "=r"(addr) : "r"((uint32_t)__cvta_generic_to_shared(&cta_best)), "r"((int)threadIdx.x));
            Top3 o;
#pragma unroll
            for (int k = 0; k < 3; ++k)
                asm volatile("ld.shared::cluster.u64 %0, [%1];" : "=l"(o.k[k]) : "r"(addr + 8 * k));
            peers[threadIdx.x] = o;
        }
        __syncthreads();
        if (part_id == 0 && threadIdx.x == 0)
            for (int peer = 1; peer < S; ++peer)
#pragma unroll
                for (int k = 0; k < 3; ++k) push(t, peers[peer].k[k]);
        // keep every CTA's shared memory alive until the first CTA has read it
        asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
    }
    if (part_id == 0 && threadIdx.x == 0) {
#pragma unroll
        for (int k = 0; k < 3; ++k) top3[(long long)r * 3 + k] = key_index(t.k[k]);
    }
}

__global__ void kap_accept_prefix_kernel(const int32_t* __restrict__ top3, const int32_t* __restrict__ row_indptr,
                                         const int32_t* __restrict__ proposed, int batch,
                                         int32_t* __restrict__ accepted, int32_t* __restrict__ next_token,
                                         int32_t* ctx_len)
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
    // commit: the K/V of the n - 1 - m rejected proposals falls off the end of the context (their
    // slots are overwritten by the next cycle's appends)
    if (ctx_len) ctx_len[b] -= n - 1 - m;
}

}  // namespace
}  // namespace kap

extern "C" kap_status kap_top3_accept(
    const float* logits, int64_t row_stride, const int32_t* row_indptr, const int32_t* proposed,
    int32_t batch, int32_t total_rows, int32_t vocab, int32_t* top3, int32_t* accepted,
    int32_t* next_token, int32_t* ctx_len, void* cuda_stream)
{
    using namespace kap;
    if (batch < 0 || total_rows < 0 || vocab < 3 || row_stride < vocab)
        return fail(KAP_ERR_INVALID_ARG, "batch %d, rows %d, vocab %d, row_stride %lld", batch, total_rows,
                    vocab, (long long)row_stride);
    if (batch == 0 || total_rows == 0) return KAP_OK;
    if (!logits || !row_indptr || !proposed || !top3 || !accepted || !next_token)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer");
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // CTAs per row: about 8K logits each, at most 8 (the portable cluster size; clusters of 16
    // measured slower here: few of them are resident at a time)
    int S = 1;
    while (S < 8 && (int64_t)vocab > (int64_t)S * 8192) S *= 2;
    static std::once_flag once;
    std::call_once(once, [] {
        cudaFuncSetAttribute(kap_top3_rows_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        cudaGetLastError();
    });
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)S; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)total_rows * (unsigned)S);
    cfg.blockDim = dim3(256);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = S > 1 ? 1 : 0;
    long long stride = row_stride;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kap_top3_rows_kernel, logits, stride, vocab, S, top3);
    if (e == cudaSuccess) {
        count_launch();
        kap_accept_prefix_kernel<<<(unsigned)((batch + 127) / 128), 128, 0, stream>>>(top3, row_indptr, proposed,
                                                                                    batch, accepted, next_token, ctx_len);
        e = cudaGetLastError();
        if (e == cudaSuccess) count_launch();
    }
    if (e != cudaSuccess) return fail(KAP_ERR_CUDA, "kap_top3_accept launch failed: %s", cudaGetErrorString(e));
    return KAP_OK;
}
