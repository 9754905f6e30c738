// Full-context verification (Section 3.2 "Full-context verification") on the fifth-generation tensor
// cores: tcgen05.mma with the accumulators in tensor memory.
//
// kap_attn_split_kernel gives every warp a 16-row tile and reads each K / V tile from shared memory
// once per row tile (ldmatrix + mma.sync); from two row tiles on (k = 8 drafts x 4 heads = 32 rows)
// the SM's shared-memory and issue bandwidth, not HBM, set the pace.  Here one thread issues, per
// batch of four pages,
//     S = Q K^T     eight  tcgen05.mma  64 x 64 x 16    (A = the Q tile, B = the four K tiles, both
//                   in shared memory, K-major, 128-byte swizzle: K exactly as the TMA copies left it)
//     O += P V      four   tcgen05.mma  64 x 128 x 16   (A = P from tensor memory, B = one V tile,
//                   MN-major, same swizzle)
// for all query rows at once: a tile is read from shared memory once, by the tensor core.  (A
// tcgen05.mma of this shape costs about 48 cycles whether N is 16 or 64 - measured - so scores are
// computed four pages at a time.)  Rows live in TMEM lanes: with 64-row tiles row r is lane
// (r % 16) + 32 (r / 16), i.e. rows 0-15 in the first 16 lanes of warp 0's quarter and rows 16-31 in
// the first 16 lanes of warp 1's; one softmax thread per row reads its 64 scores with tcgen05.ld
// and writes its 64 weights back as packed bf16 over the scores it has read.  (128-row tiles were
// tried first: twice the tensor work for the same 32 rows, and under the power cap the slower.)
//
// Roles of the four warps:
//   warps 0, 1  softmax: one query row per thread, 16 rows per warp (warp 1 only with more than 16 rows)
//   warp 2   lane 0 refills the shared-memory ring with TMA copies, a batch of four pages at a time
//   warp 3   lane 0 issues the MMAs: S of batch g + 1 is issued before O += P V of batch g, so the
//            tensor core computes the next scores while the softmax threads work on these
// The running maximum is lazy: the exponentials keep their reference m until a batch's maximum exceeds
// it by more than 8 (log2 units; weights stay below 256, exact in bf16 x fp32), and only then is O
// rescaled in tensor memory - after the previous batch's P V has completed and before this batch's is
// issued.  out = sum(p v) / sum(p) with the same rounded p in both sums, as in the other kernel.
//
// Shared memory: control block (page ids, barriers) 6 KiB, Q tile 8 KiB (32 rows; the MMA reads 64
// rows from there on, i.e. on into the ring - those rows' results are never looked at), ring of 12
// pages as four planes (K columns 0-63, K columns 64-127, V likewise) so that the K tiles of a batch
// are one contiguous 64-row operand.  Tensor memory: 256 columns per CTA (two S / P buffers of 64,
// O 128); two CTAs per SM is the residency limit of the shared memory, so the SM's 512 columns
// always suffice and tcgen05.alloc never waits.  Every wait on an mbarrier is bounded; a wait that
// runs out sets KAP_ERR_TIMEOUT, the roles drain and the CTA frees its tensor memory before it returns.
#pragma once

#include "kap_attn_kernel.cuh"

namespace kap {

constexpr int kUmmaSlots = 12;                 // ring slots of this kernel (two CTAs per SM)
constexpr int kUmmaBatch = 4;                  // pages per S product
constexpr int kUmmaRows = 32;                  // query rows per KV head this kernel takes
constexpr int kUmmaQBytes = 8192;              // Q tile: two halves of 32 rows x 128 B
constexpr int kUmmaPlaneBytes = kUmmaSlots * kHalfTileBytes;
constexpr int kTmemCols = 256;
constexpr int kTmemSP = 0, kTmemO = 128;       // S / P buffer b at kTmemSP + 64 b
constexpr float kLazyMax = 8.f;                // log2 units a batch's maximum may exceed the reference
constexpr int kUmmaIds = 1024;                 // page ids a CTA holds: the schedule's cap on pages per CTA
constexpr int kUmmaCtlBytes = 6144;            // control block; the Q tile behind it needs 1 KiB alignment
// 110 KiB: two CTAs per SM (2 x (110 + 1) KiB is what three CTAs of the split kernel take; 112 KiB did not fit)
constexpr int umma_smem_bytes() { return kUmmaCtlBytes + kUmmaQBytes + 4 * kUmmaPlaneBytes; }

struct UmmaControl {
    int32_t ids[kUmmaIds];                     // physical page ids of the item
    unsigned long long full[kUmmaSlots];       // ring slot s holds its page                         (TMA)
    unsigned long long s_ready[2];             // S buffer b holds a batch's scores                 (MMA commit)
    unsigned long long p_ready[2];             // P (over S buffer b) holds the batch's weights     (softmax warp)
    unsigned long long o_done[2];              // the P V products that read buffer b are done      (MMA commit)
    unsigned long long batch_free[kUmmaSlots / kUmmaBatch];   // ... and with them the batch's ring slots
    uint32_t tmem_base;
    int32_t timed_out;
};
static_assert(sizeof(UmmaControl) <= kUmmaCtlBytes, "control block too large");

__device__ __forceinline__ uint64_t umma_smem_desc(uint32_t addr, uint32_t lbo_bytes, uint32_t sbo_bytes) {
    return (uint64_t)((addr & 0x3FFFFu) >> 4) | (uint64_t)(lbo_bytes >> 4) << 16 | (uint64_t)(sbo_bytes >> 4) << 32 |
           1ull << 46 /* descriptor version */ | 2ull << 61 /* 128-byte swizzle */;
}
__host__ __device__ constexpr uint32_t umma_idesc(int M, int N, bool b_mn_major) {
    return 1u << 4 /* D fp32 */ | 1u << 7 /* A bf16 */ | 1u << 10 /* B bf16 */ | (b_mn_major ? 1u : 0u) << 16 |
           (uint32_t)(N >> 3) << 17 | (uint32_t)(M >> 4) << 24;
}
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :: "r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_ld16(uint32_t addr, uint32_t (&v)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(addr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
// 16 columns without the wait: several loads in flight, then one tmem_wait_ld()
__device__ __forceinline__ void tmem_ld16_nowait(uint32_t addr, uint32_t (&v)[16]) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(addr));
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_st16(uint32_t addr, const uint32_t (&v)[16]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
                 :: "r"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]),
                    "r"(v[8]), "r"(v[9]), "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]) : "memory");
}
__device__ __forceinline__ void tmem_st8(uint32_t addr, const uint32_t (&v)[8]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                 :: "r"(addr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <bool kNhd>
__global__ void __launch_bounds__(kThreads, 2)
kap_attn_umma_kernel(const __grid_constant__ CUtensorMap kv_map, const AttnParams p)
{
    // (no room for alignment slack, nor for the padding an alignment attribute would add: a kernel
    // without static shared memory gets its dynamic part at the start of the CTA's window, which is
    // 1 KiB aligned - the tiles need that - and the next lines check it)
    extern __shared__ unsigned char smem_raw[];
    unsigned char* smem_base = smem_raw;
    if (smem_u32(smem_base) & 1023u) {
        if (threadIdx.x == 0) atomicOr(p.status, 1 << KAP_ERR_DEVICE_INDEX);
        return;
    }
    UmmaControl* ub = reinterpret_cast<UmmaControl*>(smem_base);
    UmmaControl* tail = ub;                                  // (the split kernel's names for the shared fields)
    unsigned char* q_tile = smem_base + kUmmaCtlBytes;          // two halves of [32 rows][128 B], swizzled like a TMA tile
    unsigned char* ring = q_tile + kUmmaQBytes;              // planes: K cols 0-63 | K cols 64-127 | V cols 0-63 | V cols 64-127
    constexpr int n_slots = kUmmaSlots;
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    pdl_launch_dependents();

    // ---- prologue on static metadata only (work item, page list, q_indptr)
    const WorkItem item = p.items[blockIdx.x];
    int32_t* const offs = reinterpret_cast<int32_t*>(ring);
    for (int t = tid; t <= p.batch; t += kThreads) {
        offs[t] = p.list_indptr[t];
        offs[p.batch + 1 + t] = p.q_indptr[t];
    }
    __syncthreads();
    const int rows = item.n_q * p.G;                         // <= 32; row r lives in TMEM lane (r % 16) + 32 (r / 16)
    const int n_soft = rows > 16 ? 2 : 1;                    // softmax warps: 16 rows each (lanes 0-15 of the warp's TMEM quarter)
    int n_local = item.page_end - item.page_begin;
    if (n_local > kUmmaIds) {                                // the scheduler caps this kernel's slices at 1024 pages
        if (tid == 0) atomicOr(p.status, 1 << KAP_ERR_DEVICE_INDEX);
        n_local = kUmmaIds;
    }
    const int n_batches = (n_local + kUmmaBatch - 1) / kUmmaBatch;
    int32_t* const id_phys = ub->ids;
    const int64_t list0 = (int64_t)offs[item.seq] + item.page_begin;
    const int64_t list_end = offs[item.seq + 1];
    const int64_t q_row0 = offs[p.batch + 1 + item.seq];
    for (int j = tid; j < n_local; j += kThreads) {
        int32_t ph = (list0 + j) < list_end ? p.phys_pages[list0 + j] : -1;
        if (ph < 0 || ph >= p.num_pool_pages) { ph = 0; atomicOr(p.status, 1 << KAP_ERR_DEVICE_INDEX); }
        id_phys[j] = ph;
    }
    if (tid == 0) {
        for (int s = 0; s < n_slots; ++s) mbar_init(smem_u32(&tail->full[s]), 1);
        for (int g = 0; g < n_slots / kUmmaBatch; ++g) mbar_init(smem_u32(&ub->batch_free[g]), 1);
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&ub->s_ready[b]), 1);
            mbar_init(smem_u32(&ub->p_ready[b]), (uint32_t)n_soft);
            mbar_init(smem_u32(&ub->o_done[b]), 1);
        }
        tail->timed_out = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&kv_map) : "memory");
    }
    __syncwarp();
    if (warp == 0) {                                         // (two CTAs per SM x 256 of 512 columns: never waits)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     :: "r"(smem_u32(&ub->tmem_base)), "n"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the offsets in the ring were ordinary stores
    const uint32_t tmem = ub->tmem_base;
    const uint32_t lane_base = tmem + ((uint32_t)(warp * 32) << 16);

    const int rows_per_page = 2 * p.Hkv * kPageSize;
    const int v_row_off = p.Hkv * kPageSize;
    uint64_t policy;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
    auto fill = [&](int k) {                                 // page k of the item into ring slot k mod 12
        const int s = k % n_slots;
        const uint32_t bar = smem_u32(&tail->full[s]);
        const uint32_t dst = smem_u32(ring + s * kHalfTileBytes);
        mbar_expect_tx(bar, kPageHeadBytes);
        if (kNhd) {
            const int z = id_phys[k] * (2 * kPageSize);
            tma_load_3d(dst, &kv_map, 0, item.kv_head, z, bar, policy);
            tma_load_3d(dst + kUmmaPlaneBytes, &kv_map, 64, item.kv_head, z, bar, policy);
            tma_load_3d(dst + 2 * kUmmaPlaneBytes, &kv_map, 0, item.kv_head, z + kPageSize, bar, policy);
            tma_load_3d(dst + 3 * kUmmaPlaneBytes, &kv_map, 64, item.kv_head, z + kPageSize, bar, policy);
        } else {
            const int y = id_phys[k] * rows_per_page + item.kv_head * kPageSize;
            tma_load_2d(dst, &kv_map, 0, y, bar, policy);
            tma_load_2d(dst + kUmmaPlaneBytes, &kv_map, 64, y, bar, policy);
            tma_load_2d(dst + 2 * kUmmaPlaneBytes, &kv_map, 0, y + v_row_off, bar, policy);
            tma_load_2d(dst + 3 * kUmmaPlaneBytes, &kv_map, 64, y + v_row_off, bar, policy);
        }
    };
    const bool producer = warp == 2 && lane == 0;
    int filled = 0;
    if (p.early_kv && producer) {                            // pages older than the rows' own tokens: see kap_attn_split_kernel
        const int fresh_from = p.ctx_len[item.seq] - item.n_q;
        while (filled < n_slots && filled < n_local &&
               (item.page_begin + filled) * kPageSize + kPageSize - 1 < fresh_from) { fill(filled); ++filled; }
    }
    // ---- nothing produced by earlier kernels (Q, fresh KV, partial buffers) is touched above
    pdl_wait();
    const int L = p.ctx_len[item.seq];
    const uint64_t deadline = global_ns() + kWaitBudgetNs;
    // Q rows -> the Q tile (16-byte chunk c of row r goes to chunk c ^ (r & 7): the 128-byte swizzle)
    for (int idx = tid; idx < kUmmaRows * 16; idx += kThreads) {
        const int r = idx >> 4, c = idx & 15;
        uint4 x = make_uint4(0, 0, 0, 0);
        if (r < rows)
            x = __ldg(reinterpret_cast<const uint4*>(p.q + ((q_row0 + r / p.G) * p.Hq + item.kv_head * p.G + r % p.G) * kHeadDim) + c);
        *reinterpret_cast<uint4*>(q_tile + (c >> 3) * (kUmmaQBytes / 2) + r * 128 + (((c & 7) ^ (r & 7)) << 4)) = x;
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    __syncthreads();

    if (producer) {
        // ---- TMA: the rest of the first ring, then a batch's four slots again when its P V products are done
        // (one commit per batch: a commit per page costs the MMA thread more than the earlier refill gains)
        for (; filled < n_slots && filled < n_local; ++filled) fill(filled);
        for (int g = n_slots / kUmmaBatch; g < n_batches; ++g) {
            const int gb = g % (n_slots / kUmmaBatch);
            if (!mbar_wait(smem_u32(&ub->batch_free[gb]), (uint32_t)(g / (n_slots / kUmmaBatch) - 1) & 1u, deadline, &tail->timed_out)) break;
            for (int k = g * kUmmaBatch; k < min((g + 1) * kUmmaBatch, n_local); ++k) fill(k);
        }
    } else if (warp == 3 && lane == 0) {
        // ---- tensor core: S of batch g, then O += P V of batch g - 1
        constexpr uint32_t idesc_s = umma_idesc(64, kUmmaBatch * kPageSize, false), idesc_o = umma_idesc(64, kHeadDim, true);
        auto issue_pv = [&](int g) {                         // false: a wait ran out
            const int b = g & 1;
            if (!mbar_wait(smem_u32(&ub->p_ready[b]), (uint32_t)(g >> 1) & 1u, deadline, &tail->timed_out)) return false;
            tc_fence_after();
            const int cnt = min(kUmmaBatch, n_local - g * kUmmaBatch);
            for (int pg = 0; pg < cnt; ++pg) {
                const int s = (g * kUmmaBatch + pg) % n_slots;
                // V: 16 tokens (K) x 128 columns (N), N contiguous; columns 64-127 one plane further, 8 tokens = 1 KiB
                const uint32_t v_tile = smem_u32(ring + 2 * kUmmaPlaneBytes + s * kHalfTileBytes);
                umma_ts(tmem + kTmemO, tmem + kTmemSP + b * 64 + pg * 8, umma_smem_desc(v_tile, kUmmaPlaneBytes, 1024), idesc_o,
                        g > 0 || pg > 0);
            }
            umma_commit(smem_u32(&ub->o_done[b]));
            umma_commit(smem_u32(&ub->batch_free[g % (n_slots / kUmmaBatch)]));
            return true;
        };
        bool ok = true;
        for (int g = 0; g < n_batches && ok; ++g) {
            const int b = g & 1, s0 = (g * kUmmaBatch) % n_slots;
            const int cnt = min(kUmmaBatch, n_local - g * kUmmaBatch);
            for (int pg = 0; pg < cnt && ok; ++pg)
                ok = mbar_wait(smem_u32(&tail->full[s0 + pg]), (uint32_t)(g * kUmmaBatch / n_slots) & 1u, deadline, &tail->timed_out);
            // the weights of batch g - 2 lie over this S buffer: their products must be done
            if (ok && g >= 2) ok = mbar_wait(smem_u32(&ub->o_done[b]), (uint32_t)((g - 2) >> 1) & 1u, deadline, &tail->timed_out);
            if (!ok) break;
            tc_fence_after();
            // Q: 64 rows (M) x 128 columns (K); K: the batch's 64 token rows (N); 16 columns per MMA, 8 rows = 1 KiB
#pragma unroll
            for (int ks = 0; ks < 8; ++ks) {
                const uint32_t q_at = smem_u32(q_tile + (ks >> 2) * (kUmmaQBytes / 2) + (ks & 3) * 32);
                const uint32_t k_at = smem_u32(ring + (ks >> 2) * kUmmaPlaneBytes + s0 * kHalfTileBytes + (ks & 3) * 32);
                umma_ss(tmem + kTmemSP + b * 64, umma_smem_desc(q_at, 16, 1024), umma_smem_desc(k_at, 16, 1024), idesc_s, ks > 0);
            }
            umma_commit(smem_u32(&ub->s_ready[b]));
            if (g > 0) ok = issue_pv(g - 1);
        }
        if (ok) issue_pv(n_batches - 1);
    } else if (warp < n_soft) {
        // ---- softmax: one query row per thread (16 per warp), a batch of 64 scores at a time
        const int R = warp * 16 + lane;
        const bool valid = lane < 16 && R < rows;
        const int pos = L - item.n_q + (valid ? R / p.G : item.n_q - 1);   // this row's logical position
        const int full_vis_limit = L - item.n_q;
        const float sc = p.scale_log2;
        float m_ref = -INFINITY, l = 0.f;
        bool ok = true;
        for (int g = 0; g < n_batches; ++g) {
            const int b = g & 1;
            ok = mbar_wait(smem_u32(&ub->s_ready[b]), (uint32_t)(g >> 1) & 1u, deadline, &tail->timed_out);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            const int cnt = min(kUmmaBatch, n_local - g * kUmmaBatch);
            const int tok0 = (item.page_begin + g * kUmmaBatch) * kPageSize;   // first token of the batch
            float sv[kUmmaBatch * 16];
            {
                uint32_t v[kUmmaBatch][16];
#pragma unroll
                for (int pg = 0; pg < kUmmaBatch; ++pg) tmem_ld16_nowait(lane_base + kTmemSP + b * 64 + pg * 16, v[pg]);
                tmem_wait_ld();
#pragma unroll
                for (int pg = 0; pg < kUmmaBatch; ++pg)
#pragma unroll
                    for (int j = 0; j < 16; ++j) sv[pg * 16 + j] = __uint_as_float(v[pg][j]);
            }
            if (cnt < kUmmaBatch || tok0 + cnt * kPageSize - 1 > full_vis_limit) {
                // slots past the item's last page hold old pages; the causal / tail region
#pragma unroll
                for (int j = 0; j < kUmmaBatch * 16; ++j)
                    if (j >= cnt * kPageSize || tok0 + j > pos) sv[j] = -INFINITY;
                // value rows past the context's end may hold anything (even NaN): zero them
                for (int pg = 0; pg < cnt; ++pg) {
                    const int first_bad = L - (tok0 + pg * kPageSize);
                    if (first_bad < kPageSize && warp == 0) {
                        unsigned char* v_tile = ring + 2 * kUmmaPlaneBytes + ((g * kUmmaBatch + pg) % n_slots) * kHalfTileBytes;
                        if (lane < 16)
                            for (int r = max(first_bad, 0); r < kPageSize; ++r)
                                *reinterpret_cast<uint4*>(v_tile + (lane >> 3) * kUmmaPlaneBytes + r * 128 + (lane & 7) * 16) =
                                    make_uint4(0, 0, 0, 0);
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    }
                }
                __syncwarp();
            }
            float mx = sv[0];
#pragma unroll
            for (int j = 1; j < kUmmaBatch * 16; ++j) mx = fmaxf(mx, sv[j]);
            const float m_batch = mx * sc;                   // -inf when the row sees nothing of this batch
            const bool lift = m_batch > m_ref + kLazyMax;    // (always true for the row's first visible batch)
            if (__any_sync(0xffffffffu, lift)) {
                // O and l follow the new reference; all P V products issued so far must have landed
                const float m_new = lift ? m_batch : m_ref;
                const float factor = (m_new == -INFINITY) ? 1.f : ex2(m_ref - m_new);   // 0 on the first lift
                if (g > 0) {
                    ok = mbar_wait(smem_u32(&ub->o_done[(g - 1) & 1]), (uint32_t)((g - 1) >> 1) & 1u, deadline, &tail->timed_out);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    tc_fence_after();
#pragma unroll 1
                    for (int c = 0; c < kHeadDim; c += 16) {
                        uint32_t o[16];
                        tmem_ld16(lane_base + kTmemO + c, o);
#pragma unroll
                        for (int j = 0; j < 16; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * factor);
                        tmem_st16(lane_base + kTmemO + c, o);
                    }
                    tmem_wait_st();
                }
                l *= factor;
                m_ref = m_new;
            }
            const float mu = (m_ref == -INFINITY) ? 0.f : m_ref;
            // the weights go over the scores just read (columns 0-31 of the buffer; page pg: 8 columns)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 16; ++j) {
                    const int t = h * 32 + 2 * j;
                    pk[j] = pack_bf16(ex2(fmaf(sv[t], sc, -mu)), ex2(fmaf(sv[t + 1], sc, -mu)));
                    l += bf16_lo(pk[j]) + bf16_hi(pk[j]);    // the sum of the rounded weights, as P V uses them
                }
                tmem_st16(lane_base + kTmemSP + b * 64 + h * 16, pk);
            }
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&ub->p_ready[b]));
        }
        // ---- the last products, then this row's (m, l, O) to its partial slot or, alone, the result
        if (ok) {
            ok = mbar_wait(smem_u32(&ub->o_done[(n_batches - 1) & 1]), (uint32_t)((n_batches - 1) >> 1) & 1u, deadline, &tail->timed_out);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const bool single = item.n_splits == 1;
            const float inv = l > 0.f ? 1.f / l : 0.f;
            const int64_t q_row = q_row0 + (valid ? R / p.G : 0);
            const int head = item.kv_head * p.G + (valid ? R % p.G : 0);
            const int64_t prow = (int64_t)item.split * p.rows_cap + R;
#pragma unroll 1
            for (int c = 0; c < kHeadDim; c += 16) {
                uint32_t o[16];
                tmem_ld16(lane_base + kTmemO + c, o);
                if (!valid) continue;
                if (single) {
                    uint32_t w[8];
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        w[j] = pack_bf16(__uint_as_float(o[2 * j]) * inv, __uint_as_float(o[2 * j + 1]) * inv);
                    uint4* dst = reinterpret_cast<uint4*>(p.out + (q_row * p.Hq + head) * kHeadDim + c);
                    dst[0] = make_uint4(w[0], w[1], w[2], w[3]);
                    dst[1] = make_uint4(w[4], w[5], w[6], w[7]);
                } else {
                    uint4* dst = reinterpret_cast<uint4*>(p.part_o + prow * kHeadDim + c);
#pragma unroll
                    for (int j = 0; j < 4; ++j) dst[j] = make_uint4(o[4 * j], o[4 * j + 1], o[4 * j + 2], o[4 * j + 3]);
                }
            }
            if (valid) {
                if (single) {
                    if (p.lse) p.lse[q_row * p.Hq + head] = l > 0.f ? (m_ref + log2f(l)) * 0.6931471805599453f : -INFINITY;
                } else {
                    *reinterpret_cast<float2*>(p.part_ml + prow * 2) = make_float2(m_ref, l);
                }
            }
        }
    }
    if (lane == 0 && tail->timed_out) atomicOr(p.status, 1 << KAP_ERR_TIMEOUT);
    // ---- every role is done (or has given up): free the tensor memory
    tc_fence_before();
    __syncthreads();
    if (warp == 0)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(tmem), "n"(kTmemCols) : "memory");
}

}  // namespace kap
