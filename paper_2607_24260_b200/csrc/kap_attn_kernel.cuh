// Split-K paged attention for sm_100a, device code: the kernels behind kap_selected_decode_attn (Section 3.2,
// "Selected-KV proposal") and kap_verify_attn (Section 3.2, "Full-context verification") of the
// KAP paper, plus the log-sum-exp merge of the splits.
//
// One work item = a contiguous slice of one sequence's page list for one KV head, run by a
// thread-block cluster of C CTAs (C = 1: a single CTA), each of which takes an even part of it.
//   * each page's K and V rows for this KV head arrive by TMA tensor loads (cp.async.bulk.tensor,
//     128-byte swizzle) in a ring of shared-memory page slots, completion tracked by mbarriers;
//     the last warp of a warp group to finish a page refills its slot;
//   * the warps share the item's query rows in 16-row tiles (rows = n_q * G: the G query heads of
//     the KV head's group times the n_q query tokens, so every K/V byte is read from HBM once and
//     shared by all of them), compute S = Q K^T and O += P V with bf16 mma.sync tiles and fp32
//     accumulators, and keep a base-2 online softmax per row in registers;
//   * the warps' states are combined through shared memory, the cluster's CTAs reduce theirs
//     through distributed shared memory, and the result is either the final bf16 output (the
//     item is the whole list) or an un-normalised fp32 partial (m, l, O) for the merge pass.
// The proposal path is the n_q = 1 case of the same kernel; the causal rule "row j sees tokens
// t <= L - n_q + j" covers both paths.
//
// Every device-side wait is bounded: when a wait passes the CTA's deadline the kernel records
// KAP_ERR_TIMEOUT in the workspace status word and runs to its end without spinning again.
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "kap_internal.h"

namespace kap {

// ------------------------------------------------------------------------------ kernel geometry
constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxSlots = 24;                             // most page slots in the shared-memory ring
constexpr int kDefaultSlots = 8;                          // 8 slots -> 3 CTAs/SM, 12 -> 2, 24 -> 1
constexpr int kHalfTileBytes = kPageSize * 128;           // 16 tokens x 64 bf16 = 2048 B
constexpr int kTileBytes = 2 * kHalfTileBytes;            // K (or V) of one page and head: 4096 B
constexpr int kPageHeadBytes = 2 * kTileBytes;            // K + V: 8192 B
constexpr int kMaxIds = 640;                              // page ids a CTA can hold (its own share of an item)
constexpr int kScratchStride = kHeadDim + 8;              // floats per scratch row (bank spread)
constexpr uint64_t kWaitBudgetNs = 2000000000ull;         // per-CTA deadline for all waits

// Page ids of a CTA: phys[cap], logical[cap], mask[cap] packed into one array, cap = kMaxIds.  A
// cluster whose CTAs hold at most kPushIds ids and at most kPushRows query rows uses cap = kPushIds
// and the rest of the array as the landing zone of the push-style cluster reduction (see the
// epilogue): C * ceil(cells / C) <= kPushCells + 16 cells of (float4 o, float2 (m, l)) each.
constexpr int kPushIds = 256;
constexpr int kPlainIds = 1600;                           // physical ids only: the whole array
constexpr int kPushRows = 4;
constexpr int kPushCells = kPushRows * 32;                // (row, 4-column) cells of the item
constexpr int kZoneCells = kPushCells + kMaxCluster;
constexpr int kIdBytes = kMaxIds * 10;
constexpr int kZoneOff = kPushIds * 10;                   // byte offset of the landing zone
static_assert(kZoneOff % 16 == 0 && kZoneOff + kZoneCells * 24 <= kIdBytes, "landing zone must fit behind the ids");

struct SmemTail {                                         // control block in front of the ring
    alignas(16) unsigned char ids[kIdBytes];  // phys, logical (int32) and token masks (uint16)
    int32_t slot_page[kMaxSlots];             // list index of the page in each ring slot, -1 = no more
    uint32_t slot_done[kMaxSlots];            // warps that have finished with the slot's current page
    unsigned long long full[kMaxSlots];
    unsigned long long zone_full;             // completes when every peer has pushed its cells
    float m[kWarps][kRowTile];
    float l[kWarps][kRowTile];
    float cta_m[kRowTile * kMaxRowTiles];     // CTA-level state read by cluster peers
    float cta_l[kRowTile * kMaxRowTiles];
    int32_t timed_out;
};
constexpr int kTailBytes = ((int)sizeof(SmemTail) + 1023) / 1024 * 1024;   // the ring follows, 1 KiB aligned
static_assert(kTailBytes == 8192, "control block must stay within 8 KiB: 3 CTAs per SM with an 8-slot ring");
constexpr int smem_bytes_for(int slots) { return kTailBytes + slots * kPageHeadBytes + 1024; }  // + alignment slack

static_assert(kWarps * kRowTile * kScratchStride * 4 <= kDefaultSlots * kPageHeadBytes,
              "warp-combine scratch must fit in the smallest ring");

struct AttnParams {
    const __nv_bfloat16* q;          // [rows, Hq, d]
    const int32_t* q_indptr;         // [B+1] or null: sequence b owns row b
    const int32_t* list_indptr;      // [B+1]
    const int32_t* phys_pages;
    const int32_t* logical_pages;    // or null: logical page = position in the list
    const uint16_t* token_masks;     // or null: every token of a listed page is visible
    const int32_t* ctx_len;          // [B]
    const WorkItem* items;
    const MergeGroup* groups;
    float* part_o;                   // [slots][rows_cap][128]
    float* part_ml;                  // [slots][rows_cap][2]
    __nv_bfloat16* out;              // [rows, Hq, d]
    float* lse;                      // [rows, Hq] or null
    int32_t* status;
    long long num_pool_pages;
    int32_t Hq, Hkv, G, rows_cap;
    int32_t batch;                   // sequences (entries of list_indptr / q_indptr minus one)
    int32_t cluster, early_kv;       // CTAs per work item (cluster size); early KV prefetch
    int32_t ring_slots;              // page slots in the shared-memory ring (8, 12, 16 or 24)
    float scale_log2;                // sm_scale * log2(e)
#ifdef KAP_TRACE
    unsigned long long* trace;       // [8192 records][8] timestamps of this launch (debug builds)
#endif
};

#ifdef KAP_TRACE
#define KAP_TRACE_POINT(rec, slot) \
    do { if (p.trace && threadIdx.x == 0) p.trace[(size_t)(rec) * 8 + (slot)] = global_ns(); } while (0)
#else
#define KAP_TRACE_POINT(rec, slot) do { } while (0)
#endif

// ------------------------------------------------------------------------------- PTX primitives
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return (uint32_t)__cvta_generic_to_shared(p);
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ uint64_t global_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: spins until the phase completes or the CTA's deadline passes.  After the deadline
// every wait tries once and gives up, so the kernel always terminates.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, uint64_t deadline,
                                          volatile int32_t* timed_out) {
    if (mbar_try_wait(bar, parity)) return true;
    if (*timed_out) return false;
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((spin & 255u) == 0 && global_ns() > deadline) { *timed_out = 1; return false; }
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int32_t x,
                                            int32_t y, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int32_t x,
                                            int32_t y, int32_t z, uint32_t bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3, %4}], [%5], %6;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(bar), "l"(policy) : "memory");
}
__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                        uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                          uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
// D(16x8, fp32) += A(16x16, bf16, row) * B(16x8, bf16, col)
__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0,
                                         uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, "
        "{%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
__device__ __forceinline__ float bf16_lo(uint32_t v) { return __uint_as_float(v << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t v) { return __uint_as_float(v & 0xffff0000u); }
// Thread-block clusters: barrier over all threads of all CTAs of the cluster (release / acquire),
// and loads from a peer CTA's shared memory (distributed shared memory).
__device__ __forceinline__ void cluster_sync() {
    asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_arrive() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
}
__device__ __forceinline__ void cluster_wait() {
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_dsmem_f32x4(uint32_t addr, float4 v) {
    asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};"
                 ::"r"(addr), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ __forceinline__ void st_dsmem_f32x2(uint32_t addr, float a, float b) {
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(a), "f"(b) : "memory");
}
// arrive on a peer's mbarrier; orders this thread's earlier remote stores before it (cluster scope)
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// bounded like mbar_wait, for a barrier that peers of the cluster arrive on
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity, uint64_t deadline,
                                                  volatile int32_t* timed_out) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    for (uint32_t spin = 1;; ++spin) {
        if (mbar_try_wait_cluster(bar, parity)) return true;
        if ((spin & 255u) == 0 && global_ns() > deadline) { *timed_out = 1; return false; }
    }
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t cta_rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(cta_rank));
    return r;
}
__device__ __forceinline__ float ld_dsmem_f32(uint32_t addr) {
    float v;
    asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(addr));
    return v;
}
__device__ __forceinline__ float4 ld_dsmem_f32x4(uint32_t addr) {
    float4 v;
    asm volatile("ld.shared::cluster.v4.f32 {%0,%1,%2,%3}, [%4];"
                 : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(addr));
    return v;
}
// Programmatic dependent launch: let the next kernel on the stream start its prologue now ...
__device__ __forceinline__ void pdl_launch_dependents() {
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
// ... and wait for the previous kernel on the stream to have completed (memory visible).
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ------------------------------------------------------------------ merging partial softmax states
// (m in log2 units, l, O[4 columns]) states combine as
//     M = max m_i,  l = sum 2^(m_i - M) l_i,  O = sum 2^(m_i - M) O_i.
struct Merged { float m, l; float4 o; };

__device__ __forceinline__ void merge_into(Merged& r, float m, float l, const float4& o) {
    const float mn = fmaxf(r.m, m);
    const float mu = (mn == -INFINITY) ? 0.f : mn;
    const float a = ex2(r.m - mu), b = ex2(m - mu);
    r.l = r.l * a + l * b;
    r.o.x = r.o.x * a + o.x * b; r.o.y = r.o.y * a + o.y * b;
    r.o.z = r.o.z * a + o.z * b; r.o.w = r.o.w * a + o.w * b;
    r.m = mn;
}

// normalise, round to bf16 and store 4 consecutive outputs; lse in natural log
__device__ __forceinline__ void store_final(const AttnParams& p, int64_t q_row, int head, int c4,
                                            const Merged& r) {
    const float inv = r.l > 0.f ? 1.f / r.l : 0.f;
    uint2 v;
    v.x = pack_bf16(r.o.x * inv, r.o.y * inv);
    v.y = pack_bf16(r.o.z * inv, r.o.w * inv);
    *reinterpret_cast<uint2*>(p.out + (q_row * p.Hq + head) * kHeadDim + c4 * 4) = v;
    if (p.lse && c4 == 0)
        p.lse[q_row * p.Hq + head] = r.l > 0.f ? (r.m + log2f(r.l)) * 0.6931471805599453f : -INFINITY;
}

// Merge the splits of one group for one (row, 4-column) cell and write the final values.  The
// partials are read in batches of independent loads: one memory round trip per batch.
__device__ __forceinline__ void merge_group_cell(const AttnParams& p, const MergeGroup& g,
                                                 int64_t q_row0, int R, int c4) {
    constexpr int kBatch = 16;
    const int64_t base = (int64_t)g.first_item * p.rows_cap + R;
    const int64_t stride = p.rows_cap;
    Merged r; r.m = -INFINITY; r.l = 0.f; r.o = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i0 = 0; i0 < g.n_splits; i0 += kBatch) {
        float2 ml[kBatch];
        float4 o[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int i = min(i0 + j, g.n_splits - 1);
            ml[j] = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (base + i * stride) * 2));
            o[j] = __ldcg(reinterpret_cast<const float4*>(p.part_o + (base + i * stride) * kHeadDim) + c4);
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j)
            if (i0 + j < g.n_splits) merge_into(r, ml[j].x, ml[j].y, o[j]);
    }
    store_final(p, q_row0 + R / p.G, g.kv_head * p.G + R % p.G, c4, r);
}

// ------------------------------------------------------------------------------ the split kernel
// Shared-memory ring: 8 page slots of 8 KiB (K tile then V tile, each two 64-column halves in the
// TMA 128-byte swizzle).  With RT row tiles the 4 warps form 4/RT warp groups; page i of the slice
// belongs to group i mod (4/RT) and is consumed by that group's RT warps (one per row tile).  Each
// group owns 8/(4/RT) slots as a private ring; the last of its RT warps to release a slot refills
// it at once, so every group always has its whole ring in flight and no warp waits for a partner.
//
// kPush selects the cluster reduction: false = every CTA reads its peers' shared memory between two
// cluster barriers; true = every CTA pushes its cells into the owners' landing zones (few rows and
// short lists only: the host picks it when every item of the launch qualifies).
//
// kNhd selects the pool layout: false = [page][2][Hkv][P][d] ("HND": a page-head's K rows are
// contiguous; one 2-D tensor map over [rows][d]); true = [page][2][P][Hkv][d] ("NHD": token-major;
// a 3-D tensor map (d, head, token row) whose 64 x 1 x 16 box lands in the same shared-memory tile).
//
// kMode: 0 = general; 1 = push-style cluster reduction (kPush above); 2 = plain lists (kPlain: the
// caller gave neither logical page indices nor token masks - the verification path and the
// full-context fallback - so a CTA keeps only physical page ids and can hold 2.5 times as many).
template <int kMode, bool kNhd>
__global__ void __launch_bounds__(kThreads, 3)
kap_attn_split_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams p)
{
    extern __shared__ unsigned char smem_raw[];
    // the 128-byte swizzle pattern repeats every 1024 bytes: tiles must start on that boundary
    unsigned char* smem_base = reinterpret_cast<unsigned char*>(
        (reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    SmemTail* tail = reinterpret_cast<SmemTail*>(smem_base);
    unsigned char* ring = smem_base + kTailBytes;
    const int n_slots = p.ring_slots;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_launch_dependents();
    KAP_TRACE_POINT(blockIdx.x, 0);

    // ---- prologue on static metadata only (work list, page lists, q_indptr): with programmatic
    // dependent launch it overlaps the tail of the previous kernel on the stream.
    // A work item belongs to a cluster of C CTAs (C = 1: no cluster).  CTA `rank` takes an even
    // contiguous slice of the item's page list and stages only that; inside the slice the pages are
    // dealt round-robin to the CTA's warp groups: the k-th page of group g is local id
    // k * n_groups + g.
    // The prologue's global loads form a chain (work item -> list offsets -> page ids); under a
    // saturated memory system each link costs ~0.5 us, so the chain is kept to two links: the
    // offset arrays of the whole batch are copied to shared memory (the ring is still unused)
    // alongside the work-item load instead of after it.
    const int C = p.cluster, rank = blockIdx.x % C;
    const WorkItem item = p.items[blockIdx.x / C];
    int32_t* const offs = reinterpret_cast<int32_t*>(ring);  // [batch + 1] list offsets, then q offsets
    for (int t = tid; t <= p.batch; t += kThreads) {
        offs[t] = p.list_indptr[t];
        if (p.q_indptr) offs[p.batch + 1 + t] = p.q_indptr[t];
    }
    __syncthreads();
    const int rows = item.n_q * p.G;                         // valid query rows of this item
    int RT = (rows + kRowTile - 1) / kRowTile;               // row tiles: 1, 2 or 4
    if (RT == 3) RT = 4;
    const int n_groups = kWarps / RT;                        // warp groups
    const int n_item = item.page_end - item.page_begin;      // pages of the whole item
    const int slice0 = rank * (n_item / C) + min(rank, n_item % C);
    int n_local = n_item / C + (rank < n_item % C ? 1 : 0);  // pages of this CTA
    constexpr bool kPush = kMode == 1, kPlain = kMode == 2;
    constexpr int kIdCap = kPush ? kPushIds : kPlain ? kPlainIds : kMaxIds;
    if (n_local > kIdCap) {                                  // the scheduler caps a CTA's share at 512
        if (tid == 0) atomicOr(p.status, 1 << KAP_ERR_DEVICE_INDEX);
        n_local = kIdCap;
    }
    constexpr bool push = kPush;
    constexpr int cap = kIdCap;
    if (push && (C < 2 || rows > kPushRows)) {               // the host never launches this; the
        if (tid == 0) atomicOr(p.status, 1 << KAP_ERR_DEVICE_INDEX);   // landing zone would not fit
        return;                                              // (same decision in the whole cluster)
    }
    int32_t* const id_phys = reinterpret_cast<int32_t*>(tail->ids);
    int32_t* const id_logical = id_phys + cap;
    uint16_t* const id_mask = reinterpret_cast<uint16_t*>(id_phys + 2 * cap);
    const int n_cells = rows * 32;                           // (row, 4-column) cells of the item
    const int per_rank = (n_cells + C - 1) / C;              // cells whose final merge a CTA owns
    const int my_cells = max(0, min(n_cells, (rank + 1) * per_rank) - rank * per_rank);
    if (tid == 0) {
        for (int s = 0; s < n_slots; ++s) {
            mbar_init(smem_u32(&tail->full[s]), 1);
            tail->slot_done[s] = 0;
        }
        if (push) mbar_init(smem_u32(&tail->zone_full), (uint32_t)max(1, my_cells * C));
        tail->timed_out = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&kv_map) : "memory");
    }
    // first half of a cluster barrier; its second half (before the main loop) guarantees that
    // every peer has initialised its landing zone's barrier before anybody pushes
    if (push) cluster_arrive();
    const int64_t list0 = (int64_t)offs[item.seq] + item.page_begin;
    const int64_t list_end = offs[item.seq + 1];
    const int64_t q_row0 = p.q_indptr ? offs[p.batch + 1 + item.seq] : item.seq;
    for (int j = tid; j < n_local; j += kThreads) {
        const int i = slice0 + j;                            // entry of the item
        // the three loads are independent of one another: one round trip
        const bool listed = (list0 + i) < list_end;
        int32_t ph = listed ? p.phys_pages[list0 + i] : -1;
        if (ph < 0 || ph >= p.num_pool_pages) { ph = 0; atomicOr(p.status, 1 << KAP_ERR_DEVICE_INDEX); }
        id_phys[j] = ph;
        if (!kPlain) {
            id_logical[j] = listed && p.logical_pages ? p.logical_pages[list0 + i] : item.page_begin + i;
            id_mask[j] = listed && p.token_masks ? p.token_masks[list0 + i] : (uint16_t)0xFFFFu;
        }
    }
    __syncthreads();
    // the offsets in the ring were written by ordinary stores; the bulk copies that overwrite them
    // next go through the asynchronous proxy
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    KAP_TRACE_POINT(blockIdx.x, 1);

    const int depth = n_slots / n_groups;                    // ring slots per group
    const int grp = warp / RT, rt = warp % RT;
    const bool producer = (rt == 0) && (lane == 0);           // fills the group's ring at the start
    const int rows_per_page = 2 * p.Hkv * kPageSize;
    const int v_row_off = p.Hkv * kPageSize;
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    const int group_pages = (n_local - grp + n_groups - 1) / n_groups;   // pages of this warp group
    // put the group's k-th page into ring slot s, or publish "no more pages" there
    auto fill = [&](int s, int k) {
        const uint32_t bar = smem_u32(&tail->full[s]);
        const int idx = k * n_groups + grp;                  // local id
        if (k < group_pages) {
            tail->slot_page[s] = idx;
            const uint32_t dst = smem_u32(ring + s * kPageHeadBytes);
            mbar_expect_tx(bar, kPageHeadBytes);
            if (kNhd) {
                const int z = id_phys[idx] * (2 * kPageSize);            // token row of the page's K
                tma_load_3d(dst, &kv_map, 0, item.kv_head, z, bar, policy);
                tma_load_3d(dst + kHalfTileBytes, &kv_map, 64, item.kv_head, z, bar, policy);
                tma_load_3d(dst + kTileBytes, &kv_map, 0, item.kv_head, z + kPageSize, bar, policy);
                tma_load_3d(dst + kTileBytes + kHalfTileBytes, &kv_map, 64, item.kv_head, z + kPageSize, bar, policy);
            } else {
                const int y = id_phys[idx] * rows_per_page + item.kv_head * kPageSize;
                tma_load_2d(dst, &kv_map, 0, y, bar, policy);
                tma_load_2d(dst + kHalfTileBytes, &kv_map, 64, y, bar, policy);
                tma_load_2d(dst + kTileBytes, &kv_map, 0, y + v_row_off, bar, policy);
                tma_load_2d(dst + kTileBytes + kHalfTileBytes, &kv_map, 64, y + v_row_off, bar, policy);
            }
        } else {
            tail->slot_page[s] = -1;
            mbar_arrive(bar);                                // completes the phase with no bytes
        }
    };
    // Early KV prefetch: pages that hold only tokens older than the query rows' own tokens
    // (t < L - n_q) were written in earlier steps, so their loads may start before the previous
    // kernel on the stream has completed.  Pages holding the rows' own tokens, Q and the partial
    // buffers wait for it.  (What the previous kernel may do to ctx_len: advance it by at most n_q,
    // or lower it - a lowered value only means that some prefetched pages end up masked.)
    int filled = 0;
    if (p.early_kv) {
        // a hint only: if the previous kernel is still advancing ctx_len, an older (smaller) value
        // just makes fewer pages eligible; the masks use the value read after the wait
        const int L_hint = p.ctx_len[item.seq];
        if (producer) {
            const int fresh_from = L_hint - item.n_q;
            while (filled < depth) {
                const int idx = filled * n_groups + grp;
                const int lg = kPlain ? item.page_begin + slice0 + idx : id_logical[idx];
                if (filled >= group_pages || lg * kPageSize + kPageSize - 1 >= fresh_from) break;
                fill(grp * depth + filled, filled);
                ++filled;
            }
        }
    }
    // Where this lane's two query rows live (row R of the item = query token R / G, head R % G of
    // the group; null for padding rows), and an L2 prefetch of them: a hint only - L2 is coherent,
    // the loads themselves come after the wait.
    const int gid = lane >> 2, tid4 = lane & 3;
    const uint32_t* q_src[2];
    int q_tok[2];
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        const int R = rt * kRowTile + gid + half * 8;
        const bool valid = R < rows;
        q_tok[half] = valid ? R / p.G : item.n_q - 1;
        q_src[half] = valid ? reinterpret_cast<const uint32_t*>(
            p.q + ((q_row0 + q_tok[half]) * p.Hq + item.kv_head * p.G + R % p.G) * kHeadDim) : nullptr;
        if (valid && tid4 < 2)
            asm volatile("prefetch.global.L2 [%0];" ::"l"(q_src[half] + tid4 * 32) : "memory");
    }
    // ---- nothing else produced by earlier kernels (Q, fresh KV, partial buffers) is touched above
    pdl_wait();
    KAP_TRACE_POINT(blockIdx.x, 2);
    if (producer)
        for (; filled < depth; ++filled) fill(grp * depth + filled, filled);
    const int L = p.ctx_len[item.seq];
    const uint64_t deadline = global_ns() + kWaitBudgetNs;
    // second half of the prologue's cluster barrier: by now every peer has long arrived, so this
    // costs nothing here, and the epilogue may push without any further synchronisation
    if (push) cluster_wait();

    // Q fragments (A operand, 16 rows x 128) straight from global memory, zero for padding rows.
    uint32_t qf[8][4];
    int pos_row[2];                                          // logical position of rows gid, gid+8
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        pos_row[half] = L - item.n_q + q_tok[half];
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            qf[ks][half] = q_src[half] ? __ldg(q_src[half] + ks * 8 + tid4) : 0u;          // cols 16ks + 2tid4
            qf[ks][half + 2] = q_src[half] ? __ldg(q_src[half] + ks * 8 + 4 + tid4) : 0u;  // cols 16ks + 8 + 2tid4
        }
    }

    float o[16][4];
#pragma unroll
    for (int i = 0; i < 16; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_run[2] = {-INFINITY, -INFINITY};                 // running max (log2 units)
    // Row sums of the rounded weights: one more MMA per page, P times a matrix of ones, gives every
    // thread the complete sum of its two rows (the same fp32 sum of the same bf16 weights that the
    // P V product uses, so out = sum(p v) / sum(p) stays a true weighted mean).
    float l_acc[4] = {0.f, 0.f, 0.f, 0.f};                   // [0] row gid, [2] row gid + 8
    const float sc = p.scale_log2;
    const int full_vis_limit = L - item.n_q;                 // tokens <= this are visible to all rows

    // per-lane ldmatrix row addressing inside a tile (row = token, 128-byte rows, 16-byte chunk
    // index xor (row & 7) = the TMA 128-byte swizzle)
    const int lm = lane >> 3, lr = lane & 7;
    const int k_tok = ((lm >> 1) << 3) + lr, k_cbit = lm & 1;   // K: matrices (n-tile, k-half)
    const int v_tok = ((lm & 1) << 3) + lr, v_cbit = lm >> 1;   // V^T: matrices (k-half, n-tile)
    // Byte offset of this lane's ldmatrix row inside a tile for 16-byte chunk pair c (c = 0, 2, 4, 6):
    // row * 128 + (((c + cbit) ^ lr) << 4).  c is even and cbit is one bit, so (c + cbit) ^ lr
    // = c ^ (cbit ^ lr): the lane's part is a constant and the chunk pair enters as one XOR.
    const uint32_t k_lane_off = (uint32_t)(k_tok * 128 + ((k_cbit ^ lr) << 4));
    const uint32_t v_lane_off = (uint32_t)(v_tok * 128 + ((v_cbit ^ lr) << 4));
    const uint32_t ones_bf16 = 0x3F803F80u;                    // two bf16 1.0: B operand of the row-sum MMA

    // the group's ring position and barrier phase advance by counting: depth is a run-time value
    // and a division per page would cost more than the page's address arithmetic
    int ring_pos = 0;
    uint32_t parity = 0;
    for (int i = 0;; ++i) {
        const int s = grp * depth + ring_pos;
        const bool arrived = mbar_wait(smem_u32(&tail->full[s]), parity, deadline, &tail->timed_out);
        if (i == 0) KAP_TRACE_POINT(blockIdx.x, 3);
        const int page = tail->slot_page[s];
        if (page < 0 || !arrived) break;                     // the list is exhausted (or a wait ran out)
        if (++ring_pos == depth) { ring_pos = 0; parity ^= 1u; }
        const uint32_t tmask = kPlain ? 0xFFFFu : id_mask[page];
        const uint32_t kb = smem_u32(ring + s * kPageHeadBytes);
        const uint32_t vb = kb + kTileBytes;
        const int tok0 = (kPlain ? item.page_begin + slice0 + page : id_logical[page]) * kPageSize;

        // S = Q K^T for the page's 16 tokens (two n-tiles of 8)
        float sacc[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
        for (int ks = 0; ks < 8; ++ks) {
            uint32_t b0, b1, b2, b3;
            ldsm_x4(((kb + k_lane_off) ^ (uint32_t)((ks & 3) << 5)) + (ks >> 2) * kHalfTileBytes, b0, b1, b2, b3);
            mma_bf16(sacc[0], qf[ks], b0, b1);
            mma_bf16(sacc[1], qf[ks], b2, b3);
        }
        if (tok0 + kPageSize - 1 > full_vis_limit || tmask != 0xFFFFu) {
            // page reaches into the causal / tail region, or only some of its tokens are in the
            // selected union: mask per element
#pragma unroll
            for (int nt = 0; nt < 2; ++nt)
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const int slot = nt * 8 + tid4 * 2 + (e & 1);
                    if (tok0 + slot > pos_row[e >> 1] || !((tmask >> slot) & 1u)) sacc[nt][e] = -INFINITY;
                }
            // value rows past the end of the context may hold anything (even NaN): zero them
            const int first_bad = L - tok0;
            if (first_bad < kPageSize) {
                if (lane < 16) {
                    for (int r = max(first_bad, 0); r < kPageSize; ++r)
                        *reinterpret_cast<uint4*>(ring + s * kPageHeadBytes + kTileBytes
                                                  + (lane >> 3) * kHalfTileBytes + r * 128
                                                  + (lane & 7) * 16) = make_uint4(0, 0, 0, 0);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
            }
        }
        // online softmax (base 2): rows gid (e = 0,1) and gid + 8 (e = 2,3)
        float mx[2];
        mx[0] = fmaxf(fmaxf(sacc[0][0], sacc[0][1]), fmaxf(sacc[1][0], sacc[1][1]));
        mx[1] = fmaxf(fmaxf(sacc[0][2], sacc[0][3]), fmaxf(sacc[1][2], sacc[1][3]));
        float corr[2], mu[2];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
            const float mn = fmaxf(m_run[h], mx[h] * sc);
            mu[h] = (mn == -INFINITY) ? 0.f : mn;
            corr[h] = ex2(m_run[h] - mu[h]);
            m_run[h] = mn;
        }
        uint32_t pa[4];      // P as the A operand of P V (rows gid / gid+8, tokens 0-7 / 8-15)
        pa[0] = pack_bf16(ex2(fmaf(sacc[0][0], sc, -mu[0])), ex2(fmaf(sacc[0][1], sc, -mu[0])));
        pa[1] = pack_bf16(ex2(fmaf(sacc[0][2], sc, -mu[1])), ex2(fmaf(sacc[0][3], sc, -mu[1])));
        pa[2] = pack_bf16(ex2(fmaf(sacc[1][0], sc, -mu[0])), ex2(fmaf(sacc[1][1], sc, -mu[0])));
        pa[3] = pack_bf16(ex2(fmaf(sacc[1][2], sc, -mu[1])), ex2(fmaf(sacc[1][3], sc, -mu[1])));
        if (__any_sync(0xffffffffu, corr[0] != 1.f || corr[1] != 1.f)) {
#pragma unroll
            for (int n = 0; n < 16; ++n) {
                o[n][0] *= corr[0]; o[n][1] *= corr[0];
                o[n][2] *= corr[1]; o[n][3] *= corr[1];
            }
            l_acc[0] *= corr[0]; l_acc[1] *= corr[0];
            l_acc[2] *= corr[1]; l_acc[3] *= corr[1];
        }
        mma_bf16(l_acc, pa, ones_bf16, ones_bf16);
        // O += P V   (16 n-tiles of 8 output columns, two per ldmatrix)
#pragma unroll
        for (int n2 = 0; n2 < 8; ++n2) {
            uint32_t v0, v1, v2, v3;
            ldsm_x4_t(((vb + v_lane_off) ^ (uint32_t)((n2 & 3) << 5)) + (n2 >> 2) * kHalfTileBytes, v0, v1, v2, v3);
            mma_bf16(o[2 * n2], pa, v0, v1);
            mma_bf16(o[2 * n2 + 1], pa, v2, v3);
        }
        // Done with the slot.  The last of the group's RT warps to get here refills it with the
        // group's page i + depth; nobody waits for anybody.  The fences order this warp's reads
        // of the slot before the counter update and the refill's asynchronous writes after it.
        __syncwarp();
        if (lane == 0) {
            bool last = true;
            if (RT > 1) {
                __threadfence_block();
                last = atomicAdd(&tail->slot_done[s], 1u) == (uint32_t)(RT - 1);
                if (last) { tail->slot_done[s] = 0; __threadfence_block(); }
            }
            if (last) {
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                fill(s, i + depth);
            }
        }
    }
    if (lane == 0 && tail->timed_out) atomicOr(p.status, 1 << KAP_ERR_TIMEOUT);
    KAP_TRACE_POINT(blockIdx.x, 4);

    // ------------------------------------------------ combine the four warps' states, write out
    const float l_run[2] = {l_acc[0], l_acc[2]};       // complete row sums (every column of P x ones)
    __syncthreads();                                   // all tile reads done: the ring is scratch now
    float* scratch = reinterpret_cast<float*>(ring) + warp * (kRowTile * kScratchStride);
#pragma unroll
    for (int n = 0; n < 16; ++n) {                      // padding rows are never read back
        if (rt * kRowTile + gid < rows)
            *reinterpret_cast<float2*>(scratch + gid * kScratchStride + n * 8 + tid4 * 2) =
                make_float2(o[n][0], o[n][1]);
        if (rt * kRowTile + gid + 8 < rows)
            *reinterpret_cast<float2*>(scratch + (gid + 8) * kScratchStride + n * 8 + tid4 * 2) =
                make_float2(o[n][2], o[n][3]);
    }
    if (tid4 == 0) {
        tail->m[warp][gid] = m_run[0];     tail->l[warp][gid] = l_run[0];
        tail->m[warp][gid + 8] = m_run[1]; tail->l[warp][gid + 8] = l_run[1];
    }
    __syncthreads();

    float* all = reinterpret_cast<float*>(ring);
    float* m_flat = tail->cta_m;
    float* l_flat = tail->cta_l;
    const bool single = item.n_splits == 1;
    // Combine the warp groups: the CTA-level state of row R ends up in scratch row R (the region
    // of warp R / 16 of group 0, which only this cell's thread reads) and cta_m[R], cta_l[R]; with
    // one CTA per item it goes straight to global memory instead.
    KAP_TRACE_POINT(blockIdx.x, 6);
    for (int idx = tid; idx < rows * 32; idx += kThreads) {
        const int R = idx >> 5, c4 = idx & 31;
        const int t = R / kRowTile, r = R % kRowTile;
        Merged res; res.m = -INFINITY; res.l = 0.f; res.o = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int g = 0; g < n_groups; ++g) {            // warps g * RT + t hold row tile t
            const int w = g * RT + t;
            merge_into(res, tail->m[w][r], tail->l[w][r],
                       *reinterpret_cast<const float4*>(all + (w * kRowTile + r) * kScratchStride + c4 * 4));
        }
        if (C == 1) {
            if (single) {
                store_final(p, q_row0 + R / p.G, item.kv_head * p.G + R % p.G, c4, res);
            } else {
                const int64_t prow = (int64_t)item.split * p.rows_cap + R;
                *(reinterpret_cast<float4*>(p.part_o + prow * kHeadDim) + c4) = res.o;
                if (c4 == 0) *reinterpret_cast<float2*>(p.part_ml + prow * 2) = make_float2(res.m, res.l);
            }
        } else if (push) {
            // Push-style cluster reduction: the cell goes straight into the landing zone of the
            // CTA that owns it (slot: this CTA's rank), followed by an arrive on the owner's
            // barrier that orders the stores before it.  Nobody reads this CTA's shared memory, so
            // it may exit as soon as its own cells are complete.
            const int owner = idx / per_rank, slot = rank * per_rank + idx % per_rank;
            unsigned char* zone = tail->ids + kZoneOff;
            st_dsmem_f32x4(map_to_cta(smem_u32(zone + slot * 16), owner), res.o);
            st_dsmem_f32x2(map_to_cta(smem_u32(zone + kZoneCells * 16 + slot * 8), owner), res.m, res.l);
            mbar_arrive_remote(map_to_cta(smem_u32(&tail->zone_full), owner));
        } else {
            *reinterpret_cast<float4*>(all + R * kScratchStride + c4 * 4) = res.o;
            if (c4 == 0) { m_flat[R] = res.m; l_flat[R] = res.l; }
        }
    }
    if (push) {
        // owner side: cell `tid` of this CTA's share is complete once all C CTAs have pushed
        if (tid < my_cells) {
            if (mbar_wait_cluster(smem_u32(&tail->zone_full), 0, deadline, &tail->timed_out)) {
                const int idx = rank * per_rank + tid;
                const int R = idx >> 5, c4 = idx & 31;
                const unsigned char* zone = tail->ids + kZoneOff;
                Merged res; res.m = -INFINITY; res.l = 0.f; res.o = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int u = 0; u < C; ++u) {
                    const int slot = u * per_rank + tid;
                    const float2 ml = *reinterpret_cast<const float2*>(zone + kZoneCells * 16 + slot * 8);
                    merge_into(res, ml.x, ml.y, *reinterpret_cast<const float4*>(zone + slot * 16));
                }
                if (single) {
                    store_final(p, q_row0 + R / p.G, item.kv_head * p.G + R % p.G, c4, res);
                } else {
                    const int64_t prow = (int64_t)item.split * p.rows_cap + R;
                    *(reinterpret_cast<float4*>(p.part_o + prow * kHeadDim) + c4) = res.o;
                    if (c4 == 0) *reinterpret_cast<float2*>(p.part_ml + prow * 2) = make_float2(res.m, res.l);
                }
            } else {
                atomicOr(p.status, 1 << KAP_ERR_TIMEOUT);
            }
        }
    } else if (C > 1) {
        // Cluster reduction through distributed shared memory: after the first cluster barrier
        // every CTA's state is visible to its peers; rank r merges its share of the (row, column)
        // cells over all C CTAs and writes them out; the second barrier keeps every CTA's shared
        // memory alive until all peers have read it.
        cluster_sync();
        const int c_end = min(n_cells, (rank + 1) * per_rank);
        for (int idx = rank * per_rank + tid; idx < c_end; idx += kThreads) {
            const int R = idx >> 5, c4 = idx & 31;
            Merged res; res.m = -INFINITY; res.l = 0.f; res.o = make_float4(0.f, 0.f, 0.f, 0.f);
            const uint32_t o_addr = smem_u32(all + R * kScratchStride + c4 * 4);
            const uint32_t m_addr = smem_u32(m_flat + R), l_addr = smem_u32(l_flat + R);
            // four peers' states are requested before any of them is used: one round trip through
            // the cluster's shared-memory network per batch instead of one per peer
            for (int p0 = 0; p0 < C; p0 += 4) {
                float pm[4], pl[4];
                float4 po[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) {
                    const int peer = min(p0 + u, C - 1);
                    pm[u] = ld_dsmem_f32(map_to_cta(m_addr, peer));
                    pl[u] = ld_dsmem_f32(map_to_cta(l_addr, peer));
                    po[u] = ld_dsmem_f32x4(map_to_cta(o_addr, peer));
                }
#pragma unroll
                for (int u = 0; u < 4; ++u)
                    if (p0 + u < C) merge_into(res, pm[u], pl[u], po[u]);
            }
            if (single) {
                store_final(p, q_row0 + R / p.G, item.kv_head * p.G + R % p.G, c4, res);
            } else {
                const int64_t prow = (int64_t)item.split * p.rows_cap + R;
                *(reinterpret_cast<float4*>(p.part_o + prow * kHeadDim) + c4) = res.o;
                if (c4 == 0) *reinterpret_cast<float2*>(p.part_ml + prow * 2) = make_float2(res.m, res.l);
            }
        }
        cluster_sync();
    }
    KAP_TRACE_POINT(blockIdx.x, 5);
#ifdef KAP_TRACE
    if (p.trace && tid == 0) {
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        p.trace[(size_t)blockIdx.x * 8 + 7] = smid;
    }
#endif
}

// -------------------------------------------------------------------- the separate merge kernel
// grid.x = (sequence, KV head) groups that have more than one split, grid.y = blocks of 4 query
// rows; 128 threads = 4 rows x 32 four-column cells, one cell per thread.
__global__ void __launch_bounds__(128)
kap_attn_merge_kernel(const AttnParams p, const MergeGroup* merge_groups)
{
    pdl_launch_dependents();
    KAP_TRACE_POINT(4096 + blockIdx.x, 0);
    const MergeGroup g = merge_groups[blockIdx.x];          // static metadata: before the wait
    const int64_t q_row0 = p.q_indptr ? p.q_indptr[g.seq] : g.seq;
    const int R = blockIdx.y * 4 + (threadIdx.x >> 5), c4 = threadIdx.x & 31;
    pdl_wait();
    KAP_TRACE_POINT(4096 + blockIdx.x, 2);
    if (R < g.n_q * p.G) merge_group_cell(p, g, q_row0, R, c4);
    KAP_TRACE_POINT(4096 + blockIdx.x, 5);
}

// The merge pass for lists with many partial states (one long sequence cut into 50 slices): the
// next kernel on the stream waits for this pass, and one thread per output cell would read its
// states in several dependent batches.  Here eight threads share a cell: thread j merges states
// j, j + 8, ... (its loads all in flight together), then the eight running states are combined
// pairwise in a fixed order, so results do not depend on timing.  grid.x = lists, grid.y = 2 x
// query rows (a block = half a row of 32 four-column cells); a warp = 4 neighbouring cells x 8
// state lanes.
__global__ void __launch_bounds__(128)
kap_attn_merge_wide_kernel(const AttnParams p, const MergeGroup* merge_groups)
{
    pdl_launch_dependents();
    const MergeGroup g = merge_groups[blockIdx.x];          // static metadata: before the wait
    const int64_t q_row0 = p.q_indptr ? p.q_indptr[g.seq] : g.seq;
    const int R = blockIdx.y >> 1;
    const int lane = threadIdx.x & 31, sl = lane >> 2;
    const int c4 = (blockIdx.y & 1) * 16 + (threadIdx.x >> 5) * 4 + (lane & 3);
    pdl_wait();
    if (R >= g.n_q * p.G) return;                            // (the whole block: R is per block)
    constexpr int kLanes = 8, kBatch = 8;
    const int64_t base = (int64_t)g.first_item * p.rows_cap + R;
    const int64_t stride = p.rows_cap;
    Merged r; r.m = -INFINITY; r.l = 0.f; r.o = make_float4(0.f, 0.f, 0.f, 0.f);
    for (int i0 = 0; i0 < g.n_splits; i0 += kLanes * kBatch) {
        float2 ml[kBatch];
        float4 o[kBatch];
#pragma unroll
        for (int j = 0; j < kBatch; ++j) {
            const int i = min(i0 + j * kLanes + sl, g.n_splits - 1);
            ml[j] = __ldcg(reinterpret_cast<const float2*>(p.part_ml + (base + i * stride) * 2));
            o[j] = __ldcg(reinterpret_cast<const float4*>(p.part_o + (base + i * stride) * kHeadDim) + c4);
        }
#pragma unroll
        for (int j = 0; j < kBatch; ++j)
            if (i0 + j * kLanes + sl < g.n_splits) merge_into(r, ml[j].x, ml[j].y, o[j]);
    }
#pragma unroll
    for (int d = 4; d < 32; d <<= 1) {                       // state lanes differ in lane bits 2..4
        const float m2 = __shfl_xor_sync(0xffffffffu, r.m, d), l2 = __shfl_xor_sync(0xffffffffu, r.l, d);
        float4 o2;
        o2.x = __shfl_xor_sync(0xffffffffu, r.o.x, d); o2.y = __shfl_xor_sync(0xffffffffu, r.o.y, d);
        o2.z = __shfl_xor_sync(0xffffffffu, r.o.z, d); o2.w = __shfl_xor_sync(0xffffffffu, r.o.w, d);
        // both partners end with the same bits: the lower lane's state is always the left operand
        if (lane & d) { Merged t; t.m = m2; t.l = l2; t.o = o2; merge_into(t, r.m, r.l, r.o); r = t; }
        else merge_into(r, m2, l2, o2);
    }
    if (sl == 0) store_final(p, q_row0 + R / p.G, g.kv_head * p.G + R % p.G, c4, r);
}

}  // namespace kap
