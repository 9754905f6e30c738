// Host side of the split-K paged attention: workspaces, the schedule upload, tensor maps, the
// launches behind kap_selected_decode_attn and kap_verify_attn (Section 3.2 of the KAP paper:
// "Selected-KV proposal", "Full-context verification"), launch options, and the allocation-free
// entry point.  The kernels themselves are in kap_attn_kernel.cuh.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <atomic>
#include <cstring>
#include <mutex>
#include <vector>

#include "kap_internal.h"
#include "kap_attn_umma_kernel.cuh"

namespace kap {

kap_status build_schedule(int32_t batch, const int32_t* list_len, const int32_t* n_q,
                          int32_t num_q_heads, int32_t num_kv_heads, const int32_t cluster_slots[kMaxCluster],
                          const int32_t one_wave_slots[kMaxCluster], int32_t max_chunk_pages, int32_t max_items, int32_t max_rows,
                          std::vector<WorkItem>& items, std::vector<MergeGroup>& groups,
                          int32_t* max_chunk_out, int32_t* row_tiles_out, int32_t* cluster_out);

// ================================================================================= host side
namespace {
std::atomic<long long> g_launches{0};
}
void count_launch() { g_launches.fetch_add(1); }       // for the library's other translation units
int32_t* workspace_status_word(kap_workspace* ws) { return ws->d_status; }
void workspace_lists_rewritten(kap_workspace* ws) { ws->plain_next = 1; }
// A kernel that wrote several tokens per sequence into the KV pool was just enqueued on `stream`:
// the next attention launch ON THAT STREAM must not start loading "older" pages before that kernel
// has completed.  (Programmatic dependent launch only ever overlaps kernels of one stream; a launch
// on another stream is ordered against the writer by an event, i.e. completely.)  The marks are kept
// per stream so that a launch on another stream, workspace or thread cannot use one up.  When the
// small table is full, every workspace's next launch is held back once instead - never less
// cautious than needed.
namespace {
std::mutex g_bulk_mutex;
constexpr int kBulkMarks = 32;
cudaStream_t g_bulk_stream[kBulkMarks];
int g_bulk_count = 0;
unsigned long long g_bulk_overflows = 0;      // times the table was full
}
void kv_written_in_bulk(void* cuda_stream) {
    std::lock_guard<std::mutex> lock(g_bulk_mutex);
    cudaStream_t st = (cudaStream_t)cuda_stream;
    for (int i = 0; i < g_bulk_count; ++i)
        if (g_bulk_stream[i] == st) return;
    if (g_bulk_count < kBulkMarks) g_bulk_stream[g_bulk_count++] = st;
    else ++g_bulk_overflows;
}
namespace {
// true when the launch about to be enqueued on `st` follows such a write; uses the mark up
bool take_bulk_mark(kap_workspace* ws, cudaStream_t st) {
    std::lock_guard<std::mutex> lock(g_bulk_mutex);
    bool marked = ws->bulk_overflows_seen != g_bulk_overflows;
    ws->bulk_overflows_seen = g_bulk_overflows;
    for (int i = 0; i < g_bulk_count; ++i)
        if (g_bulk_stream[i] == st) {
            g_bulk_stream[i] = g_bulk_stream[--g_bulk_count];
            marked = true;
            break;
        }
    return marked;
}
}
namespace {

std::atomic<int> g_use_pdl{1};
std::atomic<int> g_max_cluster{kMaxCluster};       // largest thread-block cluster the scheduler may pick
std::atomic<int> g_early_kv{1};
std::atomic<int> g_ring_slots{kDefaultSlots};
std::atomic<int> g_ctas_per_sm{0};       // 0 = as many as fit (occupancy)
std::atomic<int> g_verify_kernel{0};     // verification launches: 0 = kap_attn_split_kernel (mma.sync), 1 = kap_attn_umma_kernel (tcgen05)
constexpr int kWideMergeSplits = 24;     // partial states per list from which the wide merge kernel pays off ...
constexpr int64_t kWideMergeRows = 1024; // ... as long as (lists x query rows) stays below this

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* f = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &f, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            f = nullptr;
        return reinterpret_cast<EncodeTiledFn>(f);
    }();
    return fn;
}

// Makes `device` current for the enclosing scope and puts the caller's device back afterwards.
struct DeviceScope {
    int prev = -1;
    cudaError_t err = cudaSuccess;
    explicit DeviceScope(int device) {
        err = cudaGetDevice(&prev);
        if (err != cudaSuccess) { prev = -1; return; }
        if (prev == device) prev = -1;            // nothing to put back
        else err = cudaSetDevice(device);
    }
    ~DeviceScope() { if (prev >= 0) cudaSetDevice(prev); }
};

// The prologue of the split kernel copies the batch's offset arrays (list offsets, and the query
// offsets on the verification path) into the still unused ring: they must fit it.
bool offsets_fit_ring(int64_t batch, bool verify, int ring_slots) {
    return (batch + 1) * (verify ? 2 : 1) * (int64_t)sizeof(int32_t) <= (int64_t)ring_slots * kPageHeadBytes;
}

#define KAP_CUDA(call)                                                                         \
    do {                                                                                       \
        cudaError_t e_ = (call);                                                               \
        if (e_ != cudaSuccess)                                                                 \
            return fail(KAP_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));         \
    } while (0)

// Tensor map over one layer's pool viewed as a 2-D bf16 matrix [pages*2*Hkv*P rows][128 cols];
// box = 16 rows x 64 columns (one half of a page-head's K or V), 128-byte swizzle.
kap_status get_tensor_map(kap_workspace* ws, const void* pool, int64_t pages, int32_t hkv,
                          const CUtensorMap** out) {
    const int32_t layout = ws->kv_layout;
    for (int i = 0; i < ws->map_count; ++i) {
        auto& s = ws->maps[i];
        if (s.base == pool && s.pages == pages && s.hkv == hkv && s.layout == layout) {
            *out = reinterpret_cast<const CUtensorMap*>(s.map);
            return KAP_OK;
        }
    }
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return fail(KAP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const uint64_t rows = (uint64_t)pages * 2 * hkv * kPageSize;
    if (rows >= (1ull << 31)) return fail(KAP_ERR_UNSUPPORTED, "pool of %lld pages is too large", (long long)pages);
    auto& slot = ws->maps[ws->map_next];
    CUresult r;
    if (layout == KAP_KV_NHD) {
        // (d, head, token row): a head's row is 256 contiguous bytes, rows of one head are
        // Hkv * 256 bytes apart; the box takes 64 columns of one head for the 16 tokens of a page
        cuuint64_t dims[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)hkv, (cuuint64_t)pages * 2 * kPageSize};
        cuuint64_t strides[2] = {(cuuint64_t)kHeadDim * 2, (cuuint64_t)hkv * kHeadDim * 2};
        cuuint32_t box[3] = {64, 1, (cuuint32_t)kPageSize};
        cuuint32_t estr[3] = {1, 1, 1};
        r = enc(reinterpret_cast<CUtensorMap*>(slot.map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3,
                const_cast<void*>(pool), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    } else {
        cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)rows};
        cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)kPageSize};
        cuuint32_t estr[2] = {1, 1};
        r = enc(reinterpret_cast<CUtensorMap*>(slot.map), CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2,
                const_cast<void*>(pool), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    }
    if (r != CUDA_SUCCESS) return fail(KAP_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
    slot.base = pool; slot.pages = pages; slot.hkv = hkv; slot.layout = layout;
    *out = reinterpret_cast<const CUtensorMap*>(slot.map);
    ws->map_next = (ws->map_next + 1) % kap_workspace::kMapSlots;
    if (ws->map_count < kap_workspace::kMapSlots) ++ws->map_count;
    return KAP_OK;
}

#ifdef KAP_TRACE
unsigned long long* g_trace = nullptr;      // [g_trace_cap launches][8192][8]
int g_trace_cap = 0, g_trace_next = 0;
#endif

kap_status launch_attention(const AttnParams& p_in, const void* pool, int64_t pages,
                            kap_workspace* ws, cudaStream_t stream) {
    if (ws->n_items == 0) return KAP_OK;
    int cur_dev = -1;
    if (cudaGetDevice(&cur_dev) != cudaSuccess || cur_dev != ws->device)
        return fail(KAP_ERR_INVALID_ARG, "the workspace belongs to device %d but device %d is current", ws->device, cur_dev);
    const CUtensorMap* map = nullptr;
    kap_status st = get_tensor_map(ws, pool, pages, p_in.Hkv, &map);
    if (st != KAP_OK) return st;
    // function attributes are per device: set them once for the workspace's device
    if (!ws->attrs_set) {
        const void* variants[6] = {(const void*)kap_attn_split_kernel<0, false>, (const void*)kap_attn_split_kernel<1, false>,
                                   (const void*)kap_attn_split_kernel<2, false>, (const void*)kap_attn_split_kernel<0, true>,
                                   (const void*)kap_attn_split_kernel<1, true>, (const void*)kap_attn_split_kernel<2, true>};
        for (const void* fn : variants) {
            cudaError_t ae = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes_for(kMaxSlots));
            if (ae != cudaSuccess) return fail(KAP_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(ae));
            cudaFuncSetAttribute(fn, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
            cudaGetLastError();
        }
        for (const void* fn : {(const void*)kap_attn_umma_kernel<false>, (const void*)kap_attn_umma_kernel<true>}) {
            cudaError_t ae = cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, umma_smem_bytes());
            if (ae != cudaSuccess) return fail(KAP_ERR_CUDA, "cudaFuncSetAttribute: %s", cudaGetErrorString(ae));
        }
        ws->attrs_set = 1;
    }

    AttnParams p = p_in;
    p.cluster = ws->cluster_size;
    p.ring_slots = ws->ring_slots;
    // after the page lists were rewritten on the device, the prologue (which reads them ahead of
    // the dependency wait) must not overlap the writer: one ordinary launch, then back to normal
    const bool use_pdl = g_use_pdl.load() && !ws->plain_next;
    ws->plain_next = 0;
    const bool after_bulk_write = take_bulk_mark(ws, stream);
    p.early_kv = (use_pdl && g_early_kv.load() && !after_bulk_write) ? 1 : 0;
#ifdef KAP_TRACE
    p.trace = (g_trace && g_trace_next < g_trace_cap) ? g_trace + (size_t)(g_trace_next++) * 8192 * 8 : nullptr;
#endif
    cudaLaunchAttribute attr[2];
    int n_attr = 0;
    if (use_pdl) {
        attr[n_attr].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[n_attr].val.programmaticStreamSerializationAllowed = 1;
        ++n_attr;
    }
    const int n_pdl_attr = n_attr;
    if (ws->cluster_size > 1) {
        attr[n_attr].id = cudaLaunchAttributeClusterDimension;
        attr[n_attr].val.clusterDim.x = (unsigned)ws->cluster_size;
        attr[n_attr].val.clusterDim.y = 1;
        attr[n_attr].val.clusterDim.z = 1;
        ++n_attr;
    }
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)ws->n_items * (unsigned)ws->cluster_size);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = ws->umma ? umma_smem_bytes() : smem_bytes_for(ws->ring_slots);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = n_attr;
    // few rows and short lists in every item (the proposal path): push-style cluster reduction
    const bool push = ws->cluster_size > 1 && ws->max_nq * p.G <= kPushRows && ws->max_chunk <= kPushIds;
    const bool nhd = ws->kv_layout == KAP_KV_NHD;
    // neither logical indices nor masks: physical ids only (longer slices fit a CTA)
    const bool plain = !push && !p.logical_pages && !p.token_masks;
    if (!plain && !push && ws->max_chunk > kMaxIds)
        return fail(KAP_ERR_INVALID_ARG, "the schedule's slices of %d pages need plain page lists (no logical "
                    "indices, no masks)", ws->max_chunk);
    if (ws->umma) {
        if (!plain || !p.q_indptr || ws->cluster_size != 1 || ws->ring_slots != kUmmaSlots)
            return fail(KAP_ERR_INVALID_ARG, "the schedule was made for the tcgen05 verification kernel: plain page lists with q_indptr only");
        if (nhd) KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_umma_kernel<true>, *map, p));
        else KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_umma_kernel<false>, *map, p));
    }
    else if (push && nhd) KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_split_kernel<1, true>, *map, p));
    else if (push) KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_split_kernel<1, false>, *map, p));
    else if (plain && nhd) KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_split_kernel<2, true>, *map, p));
    else if (plain) KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_split_kernel<2, false>, *map, p));
    else if (nhd) KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_split_kernel<0, true>, *map, p));
    else KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_split_kernel<0, false>, *map, p));
    g_launches.fetch_add(1);
    if (ws->n_merge_groups > 0) {
        const int rows = ws->max_nq * p.G;
        cfg.gridDim = dim3((unsigned)ws->n_merge_groups, (unsigned)((rows + 3) / 4));
        cfg.blockDim = dim3(128);
        cfg.dynamicSmemBytes = 0;
        cfg.numAttrs = n_pdl_attr;
        const MergeGroup* mg = ws->d_merge;
        // eight threads per output cell when the lists have many partial states and the cells are
        // few enough for that many blocks to be cheap
        if (ws->max_splits >= kWideMergeSplits && (int64_t)ws->n_merge_groups * rows <= kWideMergeRows) {
            cfg.gridDim = dim3((unsigned)ws->n_merge_groups, (unsigned)(2 * rows));
            KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_merge_wide_kernel, p, mg));
        } else {
            KAP_CUDA(cudaLaunchKernelEx(&cfg, kap_attn_merge_kernel, p, mg));
        }
        g_launches.fetch_add(1);
    }
    return KAP_OK;
}

kap_status check_shape(int32_t batch, int32_t hq, int32_t hkv, int32_t d, int32_t page,
                       const kap_workspace* ws, const void* pool, bool verify) {
    if (!ws) return fail(KAP_ERR_INVALID_ARG, "NULL workspace");
    if (d != kHeadDim || page != kPageSize)
        return fail(KAP_ERR_UNSUPPORTED, "head_dim %d / page_size %d (supported: 128 / 16)", d, page);
    if (hq <= 0 || hkv <= 0 || hq % hkv || kRowTile % (hq / hkv))
        return fail(KAP_ERR_UNSUPPORTED, "head counts %d / %d", hq, hkv);
    if (batch != ws->batch || hq != ws->num_q_heads || hkv != ws->num_kv_heads)
        return fail(KAP_ERR_INVALID_ARG, "call shape (batch %d, heads %d/%d) differs from the schedule "
                    "(batch %d, heads %d/%d)", batch, hq, hkv, ws->batch, ws->num_q_heads, ws->num_kv_heads);
    if (verify != (ws->has_nq != 0))
        return fail(KAP_ERR_INVALID_ARG, verify ? "verification needs a schedule made with n_q"
                                                : "the proposal path needs a schedule made without n_q");
    if (reinterpret_cast<uintptr_t>(pool) & 15) return fail(KAP_ERR_INVALID_ARG, "kv_pool is not 16-byte aligned");
    return KAP_OK;
}

}  // namespace
}  // namespace kap

using namespace kap;

extern "C" kap_status kap_workspace_create(kap_workspace** out, int32_t device, int32_t max_items,
                                           int32_t max_rows_per_item, int32_t max_batch) {
    if (!out) return fail(KAP_ERR_INVALID_ARG, "NULL workspace pointer");
    *out = nullptr;
    if (max_items <= 0 || max_batch <= 0 || max_rows_per_item <= 0 ||
        max_rows_per_item > kRowTile * kMaxRowTiles)
        return fail(KAP_ERR_INVALID_ARG, "workspace sizes (%d items, %d rows, %d sequences)", max_items,
                    max_rows_per_item, max_batch);
    if (!offsets_fit_ring(max_batch, true, kDefaultSlots))
        return fail(KAP_ERR_CAPACITY, "max_batch %d: a kernel stages the batch's offset arrays in %d bytes of shared "
                    "memory, which holds %d sequences", max_batch, kDefaultSlots * kPageHeadBytes,
                    kDefaultSlots * kPageHeadBytes / 8 - 1);
    DeviceScope scope(device);                    // the caller's current device is put back on return
    KAP_CUDA(scope.err);
    cudaDeviceProp prop;
    KAP_CUDA(cudaGetDeviceProperties(&prop, device));
    if (prop.major != 10)
        return fail(KAP_ERR_UNSUPPORTED, "device %d is sm_%d%d; this library is built for sm_100a only",
                    device, prop.major, prop.minor);
    auto* ws = new kap_workspace();
    ws->device = device; ws->max_items = max_items; ws->max_rows = max_rows_per_item;
    ws->max_batch = max_batch; ws->sm_count = prop.multiProcessorCount;
    const size_t max_groups = (size_t)max_items;
    cudaError_t e = cudaSuccess;
    auto dev = [&](void** p, size_t bytes) { if (e == cudaSuccess) e = cudaMalloc(p, bytes); };
    auto host = [&](void** p, size_t bytes) { if (e == cudaSuccess) e = cudaMallocHost(p, bytes); };
    dev((void**)&ws->d_items, sizeof(WorkItem) * max_items);
    dev((void**)&ws->d_groups, sizeof(MergeGroup) * max_groups);
    dev((void**)&ws->d_merge, sizeof(MergeGroup) * max_groups);
    dev((void**)&ws->d_part_o, sizeof(float) * (size_t)max_items * max_rows_per_item * kHeadDim);
    dev((void**)&ws->d_part_ml, sizeof(float) * (size_t)max_items * max_rows_per_item * 2);
    dev((void**)&ws->d_status, sizeof(int32_t));
    host((void**)&ws->h_items, sizeof(WorkItem) * max_items);
    host((void**)&ws->h_groups, sizeof(MergeGroup) * max_groups);
    host((void**)&ws->h_merge, sizeof(MergeGroup) * max_groups);
    host((void**)&ws->h_status, sizeof(int32_t));
    if (e == cudaSuccess) e = cudaMemset(ws->d_status, 0, sizeof(int32_t));
    cudaEvent_t ev = nullptr;
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
    ws->upload_event = ev;
    ws->maps = new kap_workspace::MapSlot[kap_workspace::kMapSlots]();
    if (e != cudaSuccess) {
        kap_workspace_destroy(ws);
        return fail(KAP_ERR_CUDA, "workspace allocation failed: %s", cudaGetErrorString(e));
    }
    *out = ws;
    return KAP_OK;
}

extern "C" void kap_workspace_destroy(kap_workspace* ws) {
    if (!ws) return;
    cudaFree(ws->d_items); cudaFree(ws->d_groups); cudaFree(ws->d_merge); cudaFree(ws->d_part_o);
    cudaFree(ws->d_part_ml); cudaFree(ws->d_status);
    cudaFreeHost(ws->h_items); cudaFreeHost(ws->h_groups); cudaFreeHost(ws->h_merge);
    cudaFreeHost(ws->h_status);
    if (ws->upload_event) cudaEventDestroy((cudaEvent_t)ws->upload_event);
    delete[] ws->maps;
    delete ws->schedule_key;
    delete ws;
}

extern "C" kap_status kap_schedule(kap_workspace* ws, int32_t batch, const int32_t* list_len,
                                   const int32_t* n_q, int32_t num_q_heads, int32_t num_kv_heads,
                                   int32_t max_chunk_pages, void* cuda_stream) {
    if (!ws) return fail(KAP_ERR_INVALID_ARG, "NULL workspace");
    if (batch > ws->max_batch) return fail(KAP_ERR_CAPACITY, "batch %d > workspace max_batch %d", batch, ws->max_batch);
    // The schedule depends only on these numbers: when they repeat (every decoding step of an
    // unchanged batch), the work list already on the device is the answer.
    std::vector<int32_t> key;
    key.reserve(2 * (size_t)std::max(batch, 0) + 8);
    key.push_back(batch); key.push_back(num_q_heads); key.push_back(num_kv_heads);
    key.push_back(max_chunk_pages); key.push_back(n_q != nullptr);
    key.push_back(g_ring_slots.load()); key.push_back(g_ctas_per_sm.load()); key.push_back(g_max_cluster.load());
    key.push_back(g_verify_kernel.load());
    for (int32_t b = 0; b < batch && list_len; ++b) { key.push_back(list_len[b]); key.push_back(n_q ? n_q[b] : 1); }
    if (ws->schedule_key && *ws->schedule_key == key) return KAP_OK;
    std::vector<WorkItem> items;
    std::vector<MergeGroup> groups;
    int32_t max_chunk = 0, row_tiles = 1;
    // resident CTAs per SM for the chosen ring size decide how many items make one wave;
    // clusters of 2, 4, 8 CTAs fit a few less (GPC boundaries)
    DeviceScope scope(ws->device);                // the caller's current device is put back on return
    KAP_CUDA(scope.err);
    // the tcgen05 verification kernel: 32 query rows at most, a 12-slot ring, two CTAs per SM, no clusters
    bool umma = n_q != nullptr && g_verify_kernel.load() == 1;
    for (int32_t b = 0; umma && b < batch; ++b) umma = n_q[b] * (num_q_heads / std::max(num_kv_heads, 1)) <= kUmmaRows;
    const int ring_slots = umma ? kUmmaSlots : g_ring_slots.load();
    if (!offsets_fit_ring(batch, n_q != nullptr, ring_slots))
        return fail(KAP_ERR_CAPACITY, "batch %d: the kernel stages the batch's offset arrays in its %d-slot ring "
                    "(%d bytes)", batch, ring_slots, ring_slots * kPageHeadBytes);
    const int smem = smem_bytes_for(ring_slots);
    cudaFuncSetAttribute(kap_attn_split_kernel<0, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                         smem_bytes_for(kMaxSlots));
    int occ = 0;
    cudaError_t oe;
    if (umma) {
        cudaFuncSetAttribute(kap_attn_umma_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, umma_smem_bytes());
        oe = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kap_attn_umma_kernel<false>, kThreads, umma_smem_bytes());
    } else {
        oe = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, kap_attn_split_kernel<0, false>, kThreads, smem);
    }
    if (oe != cudaSuccess || occ < 1) occ = 1;
    const int want = g_ctas_per_sm.load();
    // (the occupancy query answers 1 for any kernel that allocates tensor memory; two CTAs of 110 KiB and 256
    // columns each do become resident together - measured - so the schedule counts on two)
    const int per_sm = umma ? 2 : want > 0 ? std::min(want, occ) : occ;
    // (nothing of the workspace changes until the new schedule is complete: a failure below leaves
    // the previous schedule, ring size and cluster size in force together)
    const int32_t ctas_per_wave = per_sm * ws->sm_count;
    int32_t slots[kMaxCluster] = {ctas_per_wave};
    cudaFuncSetAttribute(kap_attn_split_kernel<0, false>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    cudaGetLastError();
    for (int c = 2; c <= kMaxCluster; ++c) {
        if (c > g_max_cluster.load() || umma) { slots[c - 1] = 0; continue; }
        cudaLaunchAttribute ca[1];
        ca[0].id = cudaLaunchAttributeClusterDimension;
        ca[0].val.clusterDim.x = (unsigned)c; ca[0].val.clusterDim.y = 1; ca[0].val.clusterDim.z = 1;
        cudaLaunchConfig_t cc{};
        cc.gridDim = dim3((unsigned)(ws->sm_count * occ / c) * (unsigned)c);
        cc.blockDim = dim3(kThreads);
        cc.dynamicSmemBytes = smem;
        cc.attrs = ca; cc.numAttrs = 1;
        int n = 0;
        if (cudaOccupancyMaxActiveClusters(&n, kap_attn_split_kernel<0, false>, &cc) != cudaSuccess) { n = 0; cudaGetLastError(); }
        slots[c - 1] = (int32_t)std::min<int64_t>((int64_t)n * per_sm / occ, ctas_per_wave / c);
    }
    // A one-wave schedule of the proposal path leaves a third of the SM's CTA slots to the next
    // kernel's early CTAs: those kernels last 10-30 us and what the early CTAs prefetch is a large
    // part of the next layer.  Verification kernels last 80-550 us; there the slots are worth more
    // than the early start (measured on the 16K configuration: 86.6 -> 84.2 us per layer).
    int32_t one_wave[kMaxCluster];
    const int keep = !n_q && per_sm >= occ && occ >= 3 ? occ - occ / 3 : per_sm;
    for (int c = 1; c <= kMaxCluster; ++c)
        one_wave[c - 1] = (int32_t)((int64_t)slots[c - 1] * keep / per_sm);
    int32_t cluster = 1;
    kap_status st = build_schedule(batch, list_len, n_q, num_q_heads, num_kv_heads, slots, one_wave,
                                   umma ? (max_chunk_pages > 0 ? std::min(max_chunk_pages, kUmmaIds) : kUmmaIds) : max_chunk_pages,
                                   ws->max_items, ws->max_rows, items, groups,
                                   &max_chunk, &row_tiles, &cluster);
    if (st != KAP_OK) return st;
    if ((int64_t)items.size() > ws->max_items || (int64_t)groups.size() > ws->max_items)
        return fail(KAP_ERR_CAPACITY, "%zu work items exceed the workspace's %d", items.size(), ws->max_items);
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    // the pinned staging buffers may still feed the previous upload
    KAP_CUDA(cudaEventSynchronize((cudaEvent_t)ws->upload_event));
    int32_t n_merge = 0;
    int64_t total_rows = 0;
    for (int32_t b = 0; b < batch; ++b) total_rows += n_q ? n_q[b] : 1;
    int32_t max_splits = 1;
    for (size_t i = 0; i < groups.size(); ++i) {
        max_splits = std::max(max_splits, groups[i].n_splits);
        ws->h_groups[i] = groups[i];
        if (groups[i].n_splits > 1) ws->h_merge[n_merge++] = groups[i];
    }
    if (!items.empty()) std::memcpy(ws->h_items, items.data(), sizeof(WorkItem) * items.size());
    if (!items.empty()) {
        KAP_CUDA(cudaMemcpyAsync(ws->d_items, ws->h_items, sizeof(WorkItem) * items.size(),
                                 cudaMemcpyHostToDevice, stream));
        KAP_CUDA(cudaMemcpyAsync(ws->d_groups, ws->h_groups, sizeof(MergeGroup) * groups.size(),
                                 cudaMemcpyHostToDevice, stream));
        if (n_merge)
            KAP_CUDA(cudaMemcpyAsync(ws->d_merge, ws->h_merge, sizeof(MergeGroup) * n_merge,
                                     cudaMemcpyHostToDevice, stream));
    }
    KAP_CUDA(cudaEventRecord((cudaEvent_t)ws->upload_event, stream));
    ws->occupancy = occ; ws->ring_slots = ring_slots; ws->ctas_per_wave = ctas_per_wave;
    ws->batch = batch; ws->n_items = (int32_t)items.size(); ws->n_groups = (int32_t)groups.size();
    ws->n_merge_groups = n_merge; ws->max_chunk = max_chunk; ws->row_tiles = row_tiles;
    ws->num_q_heads = num_q_heads; ws->num_kv_heads = num_kv_heads; ws->has_nq = n_q != nullptr;
    ws->total_rows = total_rows; ws->cluster_size = cluster; ws->umma = umma ? 1 : 0; ws->max_splits = max_splits;
    int32_t mq = 1;
    for (int32_t b = 0; b < batch; ++b) mq = std::max(mq, n_q ? n_q[b] : 1);
    ws->max_nq = mq;
    if (!ws->schedule_key) ws->schedule_key = new std::vector<int32_t>();
    *ws->schedule_key = std::move(key);
    return KAP_OK;
}

extern "C" kap_status kap_schedule_info(const kap_workspace* ws, int32_t* n_items,
                                        int32_t* n_merge_groups, int32_t* max_chunk_pages,
                                        int32_t* ctas_per_wave, int32_t* cluster_size) {
    if (!ws) return fail(KAP_ERR_INVALID_ARG, "NULL workspace");
    if (n_items) *n_items = ws->n_items;
    if (n_merge_groups) *n_merge_groups = ws->n_merge_groups;
    if (max_chunk_pages) *max_chunk_pages = ws->max_chunk;
    if (ctas_per_wave) *ctas_per_wave = ws->ctas_per_wave;
    if (cluster_size) *cluster_size = ws->cluster_size;
    return KAP_OK;
}

static AttnParams base_params(kap_workspace* ws, int32_t hq, int32_t hkv, float sm_scale,
                              int64_t num_pool_pages) {
    AttnParams p{};
    p.items = ws->d_items; p.groups = ws->d_groups; p.part_o = ws->d_part_o;
    p.part_ml = ws->d_part_ml; p.status = ws->d_status;
    p.num_pool_pages = num_pool_pages; p.Hq = hq; p.Hkv = hkv; p.G = hq / hkv;
    p.rows_cap = ws->max_rows; p.batch = ws->batch;
    p.scale_log2 = sm_scale * 1.4426950408889634f;
    return p;
}

extern "C" kap_status kap_selected_decode_attn(
    const void* q, const void* kv_pool, int64_t num_pool_pages, const int32_t* plan_indptr,
    const int32_t* plan_phys_pages, const int32_t* plan_logical_pages,
    const uint16_t* plan_token_masks, const int32_t* ctx_len,
    int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t page_size,
    float sm_scale, void* out, float* lse, kap_workspace* ws, void* cuda_stream)
{
    kap_status st = check_shape(batch, num_q_heads, num_kv_heads, head_dim, page_size, ws, kv_pool, false);
    if (st != KAP_OK) return st;
    if (batch == 0) return KAP_OK;
    if (!q || !kv_pool || !plan_indptr || !plan_phys_pages || !ctx_len || !out || num_pool_pages <= 0)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer or empty pool");
    AttnParams p = base_params(ws, num_q_heads, num_kv_heads, sm_scale, num_pool_pages);
    p.q = (const __nv_bfloat16*)q; p.q_indptr = nullptr; p.list_indptr = plan_indptr;
    p.phys_pages = plan_phys_pages; p.logical_pages = plan_logical_pages; p.ctx_len = ctx_len;
    p.token_masks = plan_token_masks;
    p.out = (__nv_bfloat16*)out; p.lse = lse;
    return launch_attention(p, kv_pool, num_pool_pages, ws, (cudaStream_t)cuda_stream);
}

extern "C" kap_status kap_verify_attn(
    const void* q, const int32_t* q_indptr, const void* kv_pool, int64_t num_pool_pages,
    const int32_t* bt_indptr, const int32_t* bt_pages, const int32_t* ctx_len, int32_t batch,
    int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t page_size, float sm_scale,
    void* out, float* lse, kap_workspace* ws, void* cuda_stream)
{
    kap_status st = check_shape(batch, num_q_heads, num_kv_heads, head_dim, page_size, ws, kv_pool, true);
    if (st != KAP_OK) return st;
    if (batch == 0) return KAP_OK;
    if (!q || !q_indptr || !kv_pool || !bt_indptr || !bt_pages || !ctx_len || !out || num_pool_pages <= 0)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer or empty pool");
    AttnParams p = base_params(ws, num_q_heads, num_kv_heads, sm_scale, num_pool_pages);
    p.q = (const __nv_bfloat16*)q; p.q_indptr = q_indptr; p.list_indptr = bt_indptr;
    p.phys_pages = bt_pages; p.logical_pages = nullptr; p.ctx_len = ctx_len;
    p.out = (__nv_bfloat16*)out; p.lse = lse;
    return launch_attention(p, kv_pool, num_pool_pages, ws, (cudaStream_t)cuda_stream);
}

extern "C" kap_status kap_workspace_check(kap_workspace* ws, void* cuda_stream) {
    if (!ws) return fail(KAP_ERR_INVALID_ARG, "NULL workspace");
    cudaStream_t stream = (cudaStream_t)cuda_stream;
    KAP_CUDA(cudaMemcpyAsync(ws->h_status, ws->d_status, sizeof(int32_t), cudaMemcpyDeviceToHost, stream));
    KAP_CUDA(cudaMemsetAsync(ws->d_status, 0, sizeof(int32_t), stream));
    KAP_CUDA(cudaStreamSynchronize(stream));
    const int32_t s = *ws->h_status;
    if (s & (1 << KAP_ERR_TIMEOUT)) return fail(KAP_ERR_TIMEOUT, "a device-side wait ran out");
    if (s & (1 << KAP_ERR_DEVICE_INDEX)) return fail(KAP_ERR_DEVICE_INDEX, "a kernel met an out-of-range page or list index");
    return KAP_OK;
}

extern "C" kap_status kap_set_launch_options(int32_t use_pdl, int32_t early_kv, int32_t ctas_per_sm,
                                             int32_t max_cluster, int32_t ring_slots) {
    if (ring_slots >= 0 && ring_slots != 8 && ring_slots != 12 && ring_slots != 16 && ring_slots != 24)
        return fail(KAP_ERR_INVALID_ARG, "ring_slots %d (allowed: 8, 12, 16, 24)", ring_slots);
    if (ring_slots > 0) g_ring_slots.store(ring_slots);
    if (max_cluster == 0 || max_cluster > kMaxCluster)
        return fail(KAP_ERR_INVALID_ARG, "max_cluster %d (allowed: 1 .. %d)", max_cluster, kMaxCluster);
    if (use_pdl >= 0) g_use_pdl.store(use_pdl ? 1 : 0);
    if (early_kv >= 0) g_early_kv.store(early_kv ? 1 : 0);
    if (ctas_per_sm >= 0) g_ctas_per_sm.store(ctas_per_sm);
    if (max_cluster > 0) g_max_cluster.store(max_cluster);
    return KAP_OK;
}

extern "C" kap_status kap_set_verify_kernel(int32_t kernel) {
    if (kernel != 0 && kernel != 1) return fail(KAP_ERR_INVALID_ARG, "kernel %d (0 = mma.sync, 1 = tcgen05)", kernel);
    g_verify_kernel.store(kernel);
    return KAP_OK;
}

extern "C" kap_status kap_workspace_set_kv_layout(kap_workspace* ws, int32_t kv_layout) {
    if (!ws) return fail(KAP_ERR_INVALID_ARG, "NULL workspace");
    if (kv_layout != KAP_KV_HND && kv_layout != KAP_KV_NHD)
        return fail(KAP_ERR_INVALID_ARG, "kv_layout %d (KAP_KV_HND = 0, KAP_KV_NHD = 1)", kv_layout);
    ws->kv_layout = kv_layout;
    return KAP_OK;
}

extern "C" int64_t kap_launch_count(void) { return g_launches.load(); }

#ifdef KAP_TRACE
// Debug builds only: device-side timestamps per CTA.  Launch l writes records [l][cta][8].
extern "C" int kap_debug_trace_begin(int launches) {
    if (g_trace) cudaFree(g_trace);
    g_trace = nullptr;
    g_trace_cap = launches; g_trace_next = 0;
    if (cudaMalloc((void**)&g_trace, (size_t)launches * 8192 * 8 * 8) != cudaSuccess) return 1;
    cudaMemset(g_trace, 0, (size_t)launches * 8192 * 8 * 8);
    return 0;
}
extern "C" int kap_debug_trace_read(unsigned long long* host, int launches) {
    cudaDeviceSynchronize();
    return cudaMemcpy(host, g_trace, (size_t)launches * 8192 * 8 * 8, cudaMemcpyDeviceToHost) != cudaSuccess;
}
#endif

// ============================================================ allocation-free proposal attention
// kap_selected_decode_attn_static: the proposal-path attention for callers that must not allocate
// device memory.  Everything the split-K kernels need beyond the caller's inputs and outputs (the
// work list, the merge map, the partial results, the status word) lives in one file-scope device
// array of fixed size, so the call makes no cudaMalloc / cudaFree and needs no kap_workspace.
namespace kap {
namespace {

constexpr size_t kStaticScratchBytes = 4u << 20;            // 4 MiB per GPU that loads the library
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_static_mutex;
unsigned char* g_static_ptr[kMaxDevices] = {};              // device address of the array, per device
bool g_static_ready[kMaxDevices] = {};

// Layout of the array for one call: [status word, padded to 256 B][items][groups][part_ml][part_o]
struct StaticLayout {
    size_t items_off, groups_off, ml_off, o_off, total;
};
StaticLayout static_layout(int64_t n_items, int64_t n_groups, int rows) {
    auto up = [](size_t v) { return (v + 255) & ~size_t(255); };
    StaticLayout l;
    l.items_off = 256;
    l.groups_off = up(l.items_off + sizeof(WorkItem) * (size_t)n_items);
    l.ml_off = up(l.groups_off + sizeof(MergeGroup) * (size_t)n_groups);
    l.o_off = up(l.ml_off + sizeof(float) * 2 * (size_t)rows * (size_t)n_items);
    l.total = up(l.o_off + sizeof(float) * (size_t)kHeadDim * (size_t)rows * (size_t)n_items);
    return l;
}

// Every (sequence, KV head) gets exactly `splits` work items of near-equal length (some may be
// empty when the list is shorter than `splits`); item and partial slot (seq * Hkv + g) * splits + s.
// A slice longer than `slice_cap` pages (what one CTA of the attention kernel can hold) is cut to
// slice_cap and reported in *status (1 << KAP_ERR_CAPACITY): the pages beyond the cut are not
// attended to, so the caller must treat the output as invalid.
__global__ void kap_static_build_items_kernel(const int32_t* __restrict__ list_indptr, int batch,
                                              int hkv, int splits, int slice_cap, WorkItem* items,
                                              MergeGroup* groups, int32_t* status) {
    const int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= batch * hkv * splits) return;
    const int s = idx % splits, grp = idx / splits, g = grp % hkv, b = grp / hkv;
    const int n = max(list_indptr[b + 1] - list_indptr[b], 0);
    const int base = n / splits, rem = n % splits;
    WorkItem it;
    it.seq = b; it.kv_head = g;
    it.page_begin = s * base + min(s, rem);
    it.page_end = it.page_begin + base + (s < rem ? 1 : 0);
    if (it.page_end - it.page_begin > slice_cap) {
        it.page_end = it.page_begin + slice_cap;
        atomicOr(status, 1 << KAP_ERR_CAPACITY);
    }
    it.group = grp; it.split = idx; it.n_splits = splits; it.n_q = 1;
    items[idx] = it;
    if (s == 0) {
        MergeGroup mg;
        mg.seq = b; mg.kv_head = g; mg.first_item = idx; mg.n_splits = splits; mg.n_q = 1;
        mg.pad[0] = mg.pad[1] = mg.pad[2] = 0;
        groups[grp] = mg;
    }
}

}  // namespace
}  // namespace kap

extern "C" kap_status kap_selected_decode_attn_static(
    const void* q, const void* kv_pool, int64_t num_pool_pages, const int32_t* plan_indptr,
    const int32_t* plan_phys_pages, const int32_t* plan_logical_pages, const int32_t* ctx_len,
    int32_t batch, int32_t num_q_heads, int32_t num_kv_heads, int32_t head_dim, int32_t page_size,
    float sm_scale, int32_t num_splits, void* out, float* lse, int32_t* device_status,
    void* cuda_stream)
{
    if (head_dim != kHeadDim || page_size != kPageSize)
        return fail(KAP_ERR_UNSUPPORTED, "head_dim %d / page_size %d (supported: 128 / 16)", head_dim, page_size);
    if (num_q_heads <= 0 || num_kv_heads <= 0 || num_q_heads % num_kv_heads ||
        kRowTile % (num_q_heads / num_kv_heads))
        return fail(KAP_ERR_UNSUPPORTED, "head counts %d / %d", num_q_heads, num_kv_heads);
    if (batch < 0 || num_splits < 1) return fail(KAP_ERR_INVALID_ARG, "batch %d / num_splits %d", batch, num_splits);
    if (batch == 0) return KAP_OK;
    if (!offsets_fit_ring(batch, false, kDefaultSlots))
        return fail(KAP_ERR_CAPACITY, "batch %d: the kernel stages the batch's offsets in %d bytes of shared memory",
                    batch, kDefaultSlots * kPageHeadBytes);
    if (!q || !kv_pool || !plan_indptr || !plan_phys_pages || !ctx_len || !out || num_pool_pages <= 0)
        return fail(KAP_ERR_INVALID_ARG, "NULL pointer or empty pool");
    if (reinterpret_cast<uintptr_t>(kv_pool) & 15) return fail(KAP_ERR_INVALID_ARG, "kv_pool is not 16-byte aligned");
    const int rows = num_q_heads / num_kv_heads;
    const int64_t n_groups = (int64_t)batch * num_kv_heads;
    const int64_t n_items = n_groups * num_splits;
    const StaticLayout lay = static_layout(n_items, n_groups, rows);
    if (n_items > (1 << 20) || lay.total > kStaticScratchBytes)
        return fail(KAP_ERR_CAPACITY,
                    "batch %d x %d KV heads x %d splits needs %zu bytes of scratch; the built-in array holds %zu "
                    "(use fewer splits or the workspace entry point)",
                    batch, num_kv_heads, num_splits, lay.total, kStaticScratchBytes);

    // one-time set-up per device: the array's name is only a host-side handle, the kernels need
    // its device address on the device that is current now
    int dev = -1;
    KAP_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kMaxDevices) return fail(KAP_ERR_UNSUPPORTED, "device index %d", dev);
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_ready[dev]) {
            void* ptr = nullptr;
            KAP_CUDA(cudaGetSymbolAddress(&ptr, g_static_scratch));
            KAP_CUDA(cudaFuncSetAttribute(kap_attn_split_kernel<0, false>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          smem_bytes_for(kMaxSlots)));
            KAP_CUDA(cudaFuncSetAttribute(kap_attn_split_kernel<2, false>,
                                          cudaFuncAttributeMaxDynamicSharedMemorySize,
                                          smem_bytes_for(kMaxSlots)));
            g_static_ptr[dev] = static_cast<unsigned char*>(ptr);
            g_static_ready[dev] = true;
        }
    }
    unsigned char* base = g_static_ptr[dev];
    cudaStream_t stream = (cudaStream_t)cuda_stream;

    // tensor map on the stack (no cache, no heap)
    EncodeTiledFn enc = encode_tiled_fn();
    if (!enc) return fail(KAP_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    const uint64_t pool_rows = (uint64_t)num_pool_pages * 2 * num_kv_heads * kPageSize;
    if (pool_rows >= (1ull << 31)) return fail(KAP_ERR_UNSUPPORTED, "pool of %lld pages is too large", (long long)num_pool_pages);
    alignas(64) CUtensorMap map;
    {
        cuuint64_t dims[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)pool_rows};
        cuuint64_t strides[1] = {(cuuint64_t)kHeadDim * 2};
        cuuint32_t box[2] = {64, (cuuint32_t)kPageSize};
        cuuint32_t estr[2] = {1, 1};
        CUresult r = enc(&map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(kv_pool), dims,
                         strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                         CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return fail(KAP_ERR_CUDA, "cuTensorMapEncodeTiled failed with %d", (int)r);
    }

    AttnParams p{};
    p.q = (const __nv_bfloat16*)q; p.q_indptr = nullptr; p.list_indptr = plan_indptr;
    p.phys_pages = plan_phys_pages; p.logical_pages = plan_logical_pages; p.ctx_len = ctx_len;
    p.items = reinterpret_cast<const WorkItem*>(base + lay.items_off);
    p.groups = reinterpret_cast<const MergeGroup*>(base + lay.groups_off);
    p.part_ml = reinterpret_cast<float*>(base + lay.ml_off);
    p.part_o = reinterpret_cast<float*>(base + lay.o_off);
    p.out = (__nv_bfloat16*)out; p.lse = lse;
    p.status = reinterpret_cast<int32_t*>(base);
    p.num_pool_pages = num_pool_pages; p.Hq = num_q_heads; p.Hkv = num_kv_heads; p.G = rows;
    p.rows_cap = rows; p.batch = batch; p.cluster = 1; p.early_kv = 0; p.ring_slots = kDefaultSlots;
    p.scale_log2 = sm_scale * 1.4426950408889634f;
#ifdef KAP_TRACE
    p.trace = nullptr;
#endif

    // the array keeps the previous call's contents: the status word must start at zero; the work
    // list and merge map are rewritten in full below, and every partial slot that the merge reads
    // is written by this call's split kernel first
    KAP_CUDA(cudaMemsetAsync(base, 0, 256, stream));
    const int threads = 128;
    // without logical indices the kernel keeps physical page ids only and a CTA holds 2.5 times
    // as many of them
    const bool plain = plan_logical_pages == nullptr;
    kap_static_build_items_kernel<<<(unsigned)((n_items + threads - 1) / threads), threads, 0, stream>>>(
        plan_indptr, batch, num_kv_heads, num_splits, plain ? kPlainIds : kMaxIds,
        reinterpret_cast<WorkItem*>(base + lay.items_off),
        reinterpret_cast<MergeGroup*>(base + lay.groups_off), reinterpret_cast<int32_t*>(base));
    KAP_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    // ordinary launches: the work list was written by the kernel just before, so the split kernel
    // must not start early
    if (plain)
        kap_attn_split_kernel<2, false><<<(unsigned)n_items, kThreads, smem_bytes_for(kDefaultSlots), stream>>>(map, p);
    else
        kap_attn_split_kernel<0, false><<<(unsigned)n_items, kThreads, smem_bytes_for(kDefaultSlots), stream>>>(map, p);
    KAP_CUDA(cudaGetLastError());
    g_launches.fetch_add(1);
    if (num_splits > 1) {
        kap_attn_merge_kernel<<<dim3((unsigned)n_groups, (unsigned)((rows + 3) / 4)), 128, 0, stream>>>(p, p.groups);
        KAP_CUDA(cudaGetLastError());
        g_launches.fetch_add(1);
    }
    if (device_status)
        KAP_CUDA(cudaMemcpyAsync(device_status, base, sizeof(int32_t), cudaMemcpyDeviceToDevice, stream));
    return KAP_OK;
}
