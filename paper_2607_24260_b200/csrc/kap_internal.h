// Internal declarations shared by the library's translation units (not part of the C ABI).
#pragma once
#include <cstdarg>
#include <cstdint>
#include <cstdio>
#include <vector>

#include "kap.h"

namespace kap {

// Sets the thread-local error text and returns `st` (so call sites can `return fail(...)`).
kap_status fail(kap_status st, const char* fmt, ...);

constexpr int kHeadDim = 128;    // d
constexpr int kPageSize = 16;    // P
constexpr int kRowTile = 16;     // query rows one warp carries (one MMA M tile)
constexpr int kMaxRowTiles = 4;  // => at most 64 rows per (sequence, KV head)
constexpr int kMaxCluster = 16;  // largest thread-block cluster (sizes above 8 are non-portable)

// One CTA's share of the work: a contiguous slice of one sequence's page list for one KV head.
struct WorkItem {
    int32_t seq;          // sequence index
    int32_t kv_head;      // KV head g
    int32_t page_begin;   // slice [page_begin, page_end) relative to the sequence's list start
    int32_t page_end;
    int32_t group;        // index of the (seq, kv_head) group this item belongs to
    int32_t split;        // index of this item among its group's splits
    int32_t n_splits;     // splits of the group; 1 => the item writes the final output itself
    int32_t n_q;          // query rows of the sequence (1 for the proposal path)
};

// One (sequence, KV head) whose splits must be merged.
struct MergeGroup {
    int32_t seq;
    int32_t kv_head;
    int32_t first_item;   // its items are first_item .. first_item + n_splits - 1
    int32_t n_splits;
    int32_t n_q;
    int32_t pad[3];
};

}  // namespace kap

struct kap_workspace {
    int32_t device = 0;
    int32_t max_items = 0, max_rows = 0, max_batch = 0;
    int32_t sm_count = 0, occupancy = 1, attrs_set = 0;
    int32_t cluster_size = 1, max_nq = 1, ring_slots = 8;   // of the last schedule
    // last schedule
    int32_t batch = 0, n_items = 0, n_groups = 0, n_merge_groups = 0, max_chunk = 0;
    int32_t max_splits = 1;                  // most partial states any list of the schedule has
    int32_t umma = 0;                        // the schedule was made for kap_attn_umma_kernel (tcgen05)
    int32_t ctas_per_wave = 0, row_tiles = 1, num_q_heads = 0, num_kv_heads = 0;
    int32_t has_nq = 0;            // schedule was made with an n_q array (verification path)
    int32_t kv_layout = 0;         // KAP_KV_HND / KAP_KV_NHD: layout of the pools given to the attention calls
    int32_t plain_next = 0;        // the page lists were just rewritten on the device: launch the
                                   // next attention kernel as an ordinary (fully ordered) one
    int64_t total_rows = 0;        // sum over sequences of n_q
    unsigned long long bulk_overflows_seen = 0;   // see kv_written_in_bulk() in kap_attn.cu
    // host (pinned) staging and device copies
    kap::WorkItem* h_items = nullptr;
    kap::WorkItem* d_items = nullptr;
    kap::MergeGroup* h_groups = nullptr;     // every (seq, kv_head), in item order
    kap::MergeGroup* d_groups = nullptr;
    kap::MergeGroup* h_merge = nullptr;      // only the groups with n_splits > 1
    kap::MergeGroup* d_merge = nullptr;
    float* d_part_o = nullptr;               // [max_items][max_rows][128]
    float* d_part_ml = nullptr;              // [max_items][max_rows][2]   (m in log2 units, l)
    int32_t* d_status = nullptr;             // device status word
    int32_t* h_status = nullptr;             // pinned read-back
    void* upload_event = nullptr;            // cudaEvent_t: last schedule upload done
    // cached tensor maps, keyed by (pool pointer, pages, Hkv)
    struct MapSlot { const void* base; int64_t pages; int32_t hkv, layout; alignas(64) unsigned char map[128]; };
    static constexpr int kMapSlots = 64;
    MapSlot* maps = nullptr;
    int32_t map_next = 0, map_count = 0;
    std::vector<int32_t>* schedule_key = nullptr;   // inputs of the schedule held on the device
};
