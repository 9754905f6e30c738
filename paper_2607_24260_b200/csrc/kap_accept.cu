// kap_top3_accept: the verifier's acceptance rule of the KAP paper (Section 3.2, Eq. 2 and the
// Top-3 instantiation of the verification policy): a proposed token is accepted when it is among
// the target model's three highest-scoring candidates at its position; m = length of the accepted
// prefix; the next carry token is the verifier's own best candidate at the first position that
// was not accepted (the bonus position when everything was accepted).
//
// Kernel 1: a cluster of up to 8 CTAs per logits row finds the row's top 3 (value descending, index ascending on
// ties, NaN ranked below everything, -inf included) - a pure streaming reduction over the vocabulary; the
// CTAs push their candidates into the first CTA's shared memory and arrive on its mbarrier.
// Kernel 2: one thread per sequence walks its rows.
#include <cuda_runtime.h>

#include <cfloat>
#include <mutex>

#include "kap_internal.h"

namespace kap {
void count_launch();

namespace {

// A logit is ranked by an order-preserving unsigned image of its value (NaN -> 1, below -inf,
// which maps to 0x007fffff; 0 = "no candidate").  While a thread scans its share of the row - in
// ascending index order - it keeps the best three images and their indices with three compares
// and twelve selects per logit, no branches: a strictly greater image moves in, so the lower
// index stays ahead on equal values.  For the merges between threads, warps and CTAs a candidate
// becomes one 64-bit key (image in the high word, complemented index in the low word), and
// keeping the best three of those is five max / min operations.
typedef unsigned long long Key;
struct Top3 { Key k[3]; };                                     // k[0] >= k[1] >= k[2]; 0 = empty
struct Scan3 { uint32_t u0, u1, u2; int i0, i1, i2; };         // u0 >= u1 >= u2; 0 = empty

__device__ __forceinline__ uint32_t image(float v) {
    const uint32_t u = __float_as_uint(v + 0.0f);               // -0.0 and +0.0 are the same value
    return (v != v) ? 1u : (u ^ ((u >> 31) ? 0xffffffffu : 0x80000000u));
}
__device__ __forceinline__ void feed(Scan3& s, float v, int i) {
    const uint32_t u = image(v);
    const bool g0 = u > s.u0, g1 = u > s.u1, g2 = u > s.u2;
    s.u2 = g1 ? s.u1 : (g2 ? u : s.u2);  s.i2 = g1 ? s.i1 : (g2 ? i : s.i2);
    s.u1 = g0 ? s.u0 : (g1 ? u : s.u1);  s.i1 = g0 ? s.i0 : (g1 ? i : s.i1);
    s.u0 = g0 ? u : s.u0;                s.i0 = g0 ? i : s.i0;
}
__device__ __forceinline__ Key as_key(uint32_t u, int i) {
    return u ? (((Key)u << 32) | (uint32_t)~i) : 0ull;
}
__device__ __forceinline__ int key_index(Key k) { return (int)~(uint32_t)k; }
__device__ __forceinline__ void push(Top3& t, Key x) {
    const Key b0 = max(t.k[0], x), r1 = min(t.k[0], x);
    const Key b1 = max(t.k[1], r1), r2 = min(t.k[1], r1);
    t.k[0] = b0; t.k[1] = b1; t.k[2] = max(t.k[2], r2);
}
// The best three keys held anywhere in the warp, left in every lane (each lane passes its own best
// three, sorted).  Three rounds of "largest head key in the warp; its owner moves on to its next
// one": keys are unique (the index is part of them), so exactly one lane advances per round, and a
// 64-bit maximum is two 32-bit warp reductions - about a tenth of the instructions of a butterfly
// of pairwise top-3 merges.
__device__ __forceinline__ void warp_top3(Top3& t) {
    Key out[3];
#pragma unroll
    for (int r = 0; r < 3; ++r) {
        const Key head = t.k[0];
        const uint32_t hi = __reduce_max_sync(0xffffffffu, (uint32_t)(head >> 32));
        const uint32_t lo = __reduce_max_sync(0xffffffffu, (uint32_t)(head >> 32) == hi ? (uint32_t)head : 0u);
        const Key best = ((Key)hi << 32) | lo;
        out[r] = best;
        if (head == best && best != 0ull) { t.k[0] = t.k[1]; t.k[1] = t.k[2]; t.k[2] = 0ull; }
    }
    t.k[0] = out[0]; t.k[1] = out[1]; t.k[2] = out[2];
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

// grid = rows * S CTAs in clusters of S: the S CTAs of a cluster share one row (a slice of the
// vocabulary each) and the cluster's first CTA merges their candidates through distributed
// shared memory.
constexpr int kRowsThreads = 256;                  // 512 measured slower: fewer clusters are resident at a time
__global__ void __launch_bounds__(kRowsThreads)
kap_top3_rows_kernel(const float* __restrict__ logits, long long row_stride, int vocab, int S,
                     int32_t* __restrict__ top3)
{
    // the prefix kernel is launched programmatically behind this one: let it become resident now
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    const int r = blockIdx.x / S, part_id = blockIdx.x % S;
    __shared__ unsigned long long landed;           // first CTA: completes when all peers have pushed
    if (S > 1) {
        if (threadIdx.x == 0 && part_id == 0) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;"
                         ::"r"((uint32_t)__cvta_generic_to_shared(&landed)), "r"(S - 1) : "memory");
            asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        }
        asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    }
    const float* row = logits + (long long)r * row_stride;
    const int per = (vocab + S - 1) / S;
    const int lo = min(vocab, part_id * per), hi = min(vocab, lo + per);
    Scan3 sc = {0u, 0u, 0u, 0, 0, 0};
    // 16-byte loads where the slice allows it, scalar head and tail otherwise
    const int head = min(hi - lo, (int)(((16 - (reinterpret_cast<uintptr_t>(row + lo) & 15)) & 15) / 4));
    for (int i = lo + threadIdx.x; i < lo + head; i += blockDim.x) feed(sc, row[i], i);
    const int n4 = (hi - lo - head) / 4;
    const float4* row4 = reinterpret_cast<const float4*>(row + lo + head);
    constexpr int kInFlight = 8;                                      // loads in flight per thread
    for (int j0 = threadIdx.x; j0 < n4; j0 += kInFlight * blockDim.x) {
        float4 x[kInFlight];
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const int j = j0 + u * blockDim.x;
            if (j < n4) x[u] = __ldcs(row4 + j);
        }
#pragma unroll
        for (int u = 0; u < kInFlight; ++u) {
            const int j = j0 + u * blockDim.x;
            if (j < n4) {
                const int i = lo + head + 4 * j;
                feed(sc, x[u].x, i); feed(sc, x[u].y, i + 1);
                feed(sc, x[u].z, i + 2); feed(sc, x[u].w, i + 3);
            }
        }
    }
    for (int i = lo + head + 4 * n4 + threadIdx.x; i < hi; i += blockDim.x) feed(sc, row[i], i);
    Top3 t;
    t.k[0] = as_key(sc.u0, sc.i0); t.k[1] = as_key(sc.u1, sc.i1); t.k[2] = as_key(sc.u2, sc.i2);
    // warp merge, then the 8 warps through shared memory
    warp_top3(t);
    __shared__ Top3 part[kRowsThreads / 32];
    __shared__ Top3 peers[8];                       // first CTA only: the other CTAs' candidates land here
    if ((threadIdx.x & 31) == 0) part[threadIdx.x >> 5] = t;
    __syncthreads();
    // second half of the cluster barrier begun at the top: the first CTA's landing barrier is
    // initialised and every peer is running
    if (S > 1) asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
    if (threadIdx.x >= 32) return;
    // warp 0 merges the warps' candidates: lane w takes warp w's three
    const int lane = threadIdx.x;
    const int n_warps = (int)(blockDim.x >> 5);
    if (lane < n_warps) t = part[lane]; else t.k[0] = t.k[1] = t.k[2] = 0;
    warp_top3(t);                                   // every lane now holds the CTA's best three
    if (S > 1 && part_id != 0) {
        // push this CTA's three candidates into the first CTA's shared memory and arrive on its
        // barrier (the arrive orders the stores before it); nobody reads this CTA's memory
        if (lane == 0) {
            uint32_t dst, bar;
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
                         : "=r"(dst) : "r"((uint32_t)__cvta_generic_to_shared(&peers[part_id])), "r"(0));
            asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
                         : "=r"(bar) : "r"((uint32_t)__cvta_generic_to_shared(&landed)), "r"(0));
#pragma unroll
            for (int k = 0; k < 3; ++k)
                asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(dst + 8 * k), "l"(t.k[k]) : "memory");
            asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(bar) : "memory");
        }
        return;
    }
    if (S > 1) {
        // bounded wait for the S - 1 arrivals; on a time-out the row keeps what this CTA found
        const uint32_t bar = (uint32_t)__cvta_generic_to_shared(&landed);
        bool ok = false;
        const unsigned long long give_up = global_ns() + 2000000000ull;
        for (uint32_t spin = 0; !ok; ++spin) {
            uint32_t done;
            asm volatile(
                "{\n\t.reg .pred p;\n\t"
                "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], 0;\n\t"
                "selp.u32 %0, 1, 0, p;\n\t}"
                : "=r"(done) : "r"(bar) : "memory");
            ok = done != 0;
            if (!ok && (spin & 255u) == 255u && global_ns() > give_up) break;
        }
        ok = __all_sync(0xffffffffu, ok);           // the lanes decide together
        if (ok) {
            if (lane >= 1 && lane < S) t = peers[lane];
            else if (lane != 0) t.k[0] = t.k[1] = t.k[2] = 0;
            warp_top3(t);                           // S <= 8 peers
        }
    }
    if (lane == 0) {
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
    // everything above reads the caller's inputs only; top3 comes from the kernel in front
    asm volatile("griddepcontrol.wait;" ::: "memory");
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
    cfg.blockDim = dim3(kRowsThreads);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = S > 1 ? 1 : 0;
    long long stride = row_stride;
    cudaError_t e = cudaLaunchKernelEx(&cfg, kap_top3_rows_kernel, logits, stride, vocab, S, top3);
    if (e == cudaSuccess) {
        count_launch();
        cudaLaunchAttribute pa[1];
        pa[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        pa[0].val.programmaticStreamSerializationAllowed = 1;
        cudaLaunchConfig_t pc{};
        pc.gridDim = dim3((unsigned)((batch + 127) / 128));
        pc.blockDim = dim3(128);
        pc.stream = stream;
        pc.attrs = pa;
        pc.numAttrs = 1;
        const int32_t* top3_in = top3;
        e = cudaLaunchKernelEx(&pc, kap_accept_prefix_kernel, top3_in, row_indptr, proposed, batch, accepted,
                               next_token, ctx_len);
        if (e == cudaSuccess) count_launch();
    }
    if (e != cudaSuccess) return fail(KAP_ERR_CUDA, "kap_top3_accept launch failed: %s", cudaGetErrorString(e));
    return KAP_OK;
}
