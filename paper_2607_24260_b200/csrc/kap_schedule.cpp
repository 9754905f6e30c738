// Split-K work scheduling for the attention kernels (host code, no GPU).
//
// The paper (Section 3.2, "Runtime stability and fallback") asks for stable metadata shapes so
// that decode steps replay as CUDA graphs; it does not describe how one sequence's pages are
// spread over a GPU.  This file is that part: every (sequence, KV head) page list is cut into
// near-equal contiguous chunks, one chunk per thread-block cluster (whose CTAs share it evenly and
// reduce their partial results through distributed shared memory), such that the clusters fill
// the GPU's resident slots in whole waves.  The result depends only on page counts and row counts, so it is
// computed once per request shape and reused for every layer and step.
#include <algorithm>
#include <cstring>
#include <functional>
#include <numeric>
#include <vector>

#include "kap_internal.h"

namespace kap {

namespace {

// chunks needed when every list is cut into pieces of at most t pages
int64_t chunks_for(const int32_t* len, int32_t batch, int32_t hkv, int64_t t) {
    int64_t n = 0;
    for (int32_t b = 0; b < batch; ++b) n += ((int64_t)len[b] + t - 1) / t;
    return n * hkv;
}

}  // namespace

// Cost model used to pick the cluster size and the number of waves, in units of "pages streamed
// by one CTA": a CTA pays a fixed start-up / epilogue cost, a launch whose groups need more than
// one cluster pays for the separate merge pass, a cluster pays for its two cluster barriers and
// the looser placement of its CTAs (measured: about 1.6 pages per CTA of the cluster; half of
// that when the kernel can use its push-style reduction, i.e. for items of at most 4 query rows).
constexpr int64_t kFixedPages = 6;                        // + rows / 2: wider items start and end slower
constexpr int64_t kMergePassPages = 9;
constexpr int64_t kMergeBatchPages = 3;                   // per further batch of 16 partial states of one list
constexpr int64_t kLaterWavePages = 40;
constexpr int64_t kClusterPagesX5 = 8;                    // per CTA of a cluster, in fifths of a page
constexpr int64_t kPushClusterPagesX5 = 4;                // same, when the kernel reduces by pushing (<= 4 rows)
constexpr int32_t kDefaultChunkCap = 512;     // pages per CTA: the kernel's page-id buffer holds 640 entries
constexpr int32_t kPlainChunkCap = 1536;      // verification lists carry physical ids only: 1600 fit

// cluster_slots[c - 1] = clusters of c CTAs that can be resident at once (0 = size not allowed);
// one_wave_slots[c - 1] = how many of them a schedule that fits one wave may use: leaving part of
// every SM free lets the next kernel's CTAs become resident early (programmatic dependent launch)
kap_status build_schedule(int32_t batch, const int32_t* list_len, const int32_t* n_q,
                          int32_t num_q_heads, int32_t num_kv_heads, const int32_t cluster_slots[kMaxCluster],
                          const int32_t one_wave_slots[kMaxCluster],
                          int32_t max_chunk_pages, int32_t max_items, int32_t max_rows,
                          std::vector<WorkItem>& items, std::vector<MergeGroup>& groups,
                          int32_t* max_chunk_out, int32_t* row_tiles_out, int32_t* cluster_out)
{
    if (batch < 0 || (batch > 0 && !list_len)) return fail(KAP_ERR_INVALID_ARG, "bad batch / list_len");
    if (num_q_heads <= 0 || num_kv_heads <= 0 || num_q_heads % num_kv_heads)
        return fail(KAP_ERR_INVALID_ARG, "head counts %d / %d", num_q_heads, num_kv_heads);
    const int32_t G = num_q_heads / num_kv_heads;
    if (kRowTile % G) return fail(KAP_ERR_UNSUPPORTED, "group size %d must divide %d", G, kRowTile);
    if (cluster_slots[0] <= 0) return fail(KAP_ERR_INVALID_ARG, "cta_slots %d", cluster_slots[0]);
    const int32_t hard_cap = n_q ? kPlainChunkCap : kDefaultChunkCap;
    const int32_t cap = max_chunk_pages <= 0 ? hard_cap : std::min(max_chunk_pages, hard_cap);
    int32_t max_len = 0, max_nq = 1;
    for (int32_t b = 0; b < batch; ++b) {
        if (list_len[b] <= 0) return fail(KAP_ERR_INVALID_ARG, "list_len[%d] = %d <= 0", b, list_len[b]);
        const int32_t nq = n_q ? n_q[b] : 1;
        if (nq < 1) return fail(KAP_ERR_INVALID_ARG, "n_q[%d] = %d < 1", b, nq);
        max_len = std::max(max_len, list_len[b]);
        max_nq = std::max(max_nq, nq);
    }
    const int32_t rows = max_nq * G;
    if (rows > kRowTile * kMaxRowTiles)
        return fail(KAP_ERR_UNSUPPORTED, "%d query rows per KV head exceed %d", rows, kRowTile * kMaxRowTiles);
    if (rows > max_rows) return fail(KAP_ERR_CAPACITY, "%d rows per item, workspace holds %d", rows, max_rows);
    int32_t row_tiles = (rows + kRowTile - 1) / kRowTile;
    if (row_tiles == 3) row_tiles = 4;
    items.clear();
    groups.clear();
    *max_chunk_out = 0;
    *row_tiles_out = row_tiles;
    *cluster_out = 1;
    if (batch == 0) return KAP_OK;

    // A candidate schedule = a cluster size C and a number of splits per sequence.  Candidates:
    // for every allowed C and wave count W, the fewest splits that keep every chunk under the
    // smallest feasible size for C-slots * W items, then the left-over items handed to the
    // sequences with the longest chunks (so whole waves are filled); plus "one cluster per
    // (sequence, KV head)" (no merge pass).  A candidate's cost is the makespan of its items on the
    // resident cluster slots under longest-first list scheduling - which is what the hardware does
    // with CTAs handed out in index order - in pages streamed per CTA, plus the fixed costs.
    const int64_t fixed = kFixedPages + rows / 2;            // start-up + epilogue of one CTA
    const int64_t n_groups_total = (int64_t)batch * num_kv_heads;
    const int64_t item_cap = std::max<int64_t>(1, max_items);
    auto min_chunk = [&](int64_t budget) -> int64_t {
        int64_t lo = 1, hi = max_len;
        if (chunks_for(list_len, batch, num_kv_heads, hi) > budget) return -1;
        while (lo < hi) {
            const int64_t mid = (lo + hi) / 2;
            if (chunks_for(list_len, batch, num_kv_heads, mid) <= budget) hi = mid; else lo = mid + 1;
        }
        return lo;
    };
    std::vector<int32_t> splits(batch), best_splits;
    std::vector<int64_t> sizes, heap;
    int64_t best_cost = INT64_MAX;
    int32_t best_c = 1;
    auto evaluate = [&](int64_t C, int64_t slots) {
        // per-CTA chunk of each item, longest first
        sizes.clear();
        bool merge_pass = false;
        int64_t total = 0, longest = 0, most_splits = 1;
        for (int32_t b = 0; b < batch; ++b) {
            const int64_t n = splits[b], base = list_len[b] / n, rem = list_len[b] % n;
            if ((base + (rem ? 1 : 0) + C - 1) / C > cap) return;
            merge_pass |= n > 1;
            most_splits = std::max(most_splits, n);
            for (int64_t i = 0; i < n; ++i) {
                const int64_t sz = (base + (i < rem ? 1 : 0) + C - 1) / C + fixed;
                for (int32_t g = 0; g < num_kv_heads; ++g) sizes.push_back(sz);
                total += sz * num_kv_heads;
                longest = std::max(longest, sz);
            }
        }
        if ((int64_t)sizes.size() > item_cap) return;
        // (the merge pass reads a list's partial states sixteen at a time, one memory round trip each)
        const int64_t penalty = (merge_pass ? kMergePassPages + kMergeBatchPages * ((most_splits - 1) / 16) : 0) + (C > 1 ? ((rows <= 4 ? kPushClusterPagesX5 : kClusterPagesX5) * C + 4) / 5 : 0);
        if (std::max(longest, (total + slots - 1) / slots) + penalty >= best_cost) return;   // lower bound
        int64_t makespan = longest;
        if ((int64_t)sizes.size() > slots) {
            std::sort(sizes.begin(), sizes.end(), std::greater<int64_t>());
            heap.assign((size_t)slots, 0);                   // min-heap of slot finish times
            auto cmp = std::greater<int64_t>();
            for (int64_t sz : sizes) {
                std::pop_heap(heap.begin(), heap.end(), cmp);
                // a CTA that starts behind another one finds no prefetched pages and cannot hide
                // its prologue behind the previous kernel: it ramps up from an empty ring
                heap.back() += sz + (heap.back() > 0 ? kLaterWavePages : 0);
                makespan = std::max(makespan, heap.back());
                std::push_heap(heap.begin(), heap.end(), cmp);
            }
        }
        if (makespan + penalty < best_cost) { best_cost = makespan + penalty; best_c = (int32_t)C; best_splits = splits; }
    };
    static const int64_t kWaves[] = {-1, 0, 1, 2, 3, 4, 5, 6, 8, 10, 12, 16, 24, 32, 48, 64, INT32_MAX};
    for (int ci = 0; ci < kMaxCluster; ++ci) {
        const int64_t C = ci + 1, slots = cluster_slots[ci];
        if (slots <= 0) continue;
        int64_t last_budget = -1;
        for (int64_t waves : kWaves) {                       // the last entry: as many items as allowed
            // (entries <= 0: a launch that fills only a half or a quarter of a wave - short lists are
            // not worth a CTA per page and a merge pass over dozens of partial states)
            const int64_t one_wave = std::min<int64_t>(slots, one_wave_slots[ci]);
            const int64_t budget = std::min<int64_t>(item_cap, waves == -1 ? std::max<int64_t>(one_wave / 4, 1) : waves == 0 ? std::max<int64_t>(one_wave / 2, 1)
                                                               : waves == 1 ? one_wave : slots * waves);
            if (budget == last_budget) break;
            last_budget = budget;
            const int64_t t = min_chunk(budget);
            if (t <= 0) continue;
            int64_t used = 0;
            for (int32_t b = 0; b < batch; ++b) { splits[b] = (int32_t)((list_len[b] + t - 1) / t); used += (int64_t)splits[b] * num_kv_heads; }
            // hand the left-over items of the last wave to the sequences with the longest chunks
            for (int64_t left = budget - used; left >= num_kv_heads; left -= num_kv_heads) {
                int32_t arg = -1; int64_t worst = 1;
                for (int32_t b = 0; b < batch; ++b) {
                    const int64_t chunk = (list_len[b] + splits[b] - 1) / splits[b];
                    if (chunk > worst) { worst = chunk; arg = b; }
                }
                if (arg < 0) break;
                ++splits[arg];
            }
            evaluate(C, slots);
            if (t <= C) break;                               // chunks cannot get any smaller
        }
        if (n_groups_total <= item_cap) {                    // one cluster per (sequence, KV head)
            std::fill(splits.begin(), splits.end(), 1);
            evaluate(C, slots);
        }
    }
    if (best_cost == INT64_MAX)
        return fail(KAP_ERR_CAPACITY, "page lists need more than %d work items of <= %d pages per CTA",
                    max_items, cap);

    int32_t slot = 0;
    for (int32_t b = 0; b < batch; ++b) {
        const int32_t len = list_len[b];
        const int32_t n_splits = best_splits[b];
        const int32_t base = len / n_splits, rem = len % n_splits;
        for (int32_t g = 0; g < num_kv_heads; ++g) {
            MergeGroup mg{};
            mg.seq = b; mg.kv_head = g; mg.first_item = slot; mg.n_splits = n_splits;
            mg.n_q = n_q ? n_q[b] : 1;
            const int32_t group_index = (int32_t)groups.size();
            groups.push_back(mg);
            int32_t begin = 0;
            for (int32_t s = 0; s < n_splits; ++s) {
                const int32_t n = base + (s < rem ? 1 : 0);
                WorkItem it{};
                it.seq = b; it.kv_head = g; it.page_begin = begin; it.page_end = begin + n;
                it.group = group_index; it.split = slot; it.n_splits = n_splits; it.n_q = mg.n_q;
                items.push_back(it);
                *max_chunk_out = std::max(*max_chunk_out, (n + best_c - 1) / best_c);
                begin += n;
                ++slot;
            }
        }
    }
    *cluster_out = best_c;
    // longest chunks first: the hardware hands out CTAs in index order, so the tail of the last
    // wave is made of the shortest chunks.  WorkItem::split holds the item's partial-result slot
    // (group.first_item + split index), which is what keeps a group's partials contiguous.
    std::stable_sort(items.begin(), items.end(), [](const WorkItem& a, const WorkItem& c) {
        return (a.page_end - a.page_begin) > (c.page_end - c.page_begin);
    });
    return KAP_OK;
}

}  // namespace kap

// Exposed for tests and tools: the same schedule kap_schedule uploads, written to HOST arrays.
// Not a paper operation (see the file header).
extern "C" kap_status kap_schedule_host(
    int32_t batch, const int32_t* list_len, const int32_t* n_q, int32_t num_q_heads,
    int32_t num_kv_heads, int32_t cta_slots, int32_t max_cluster, int32_t max_chunk_pages,
    int32_t max_items, int32_t* items_out, int32_t* n_items, int32_t* n_merge_groups,
    int32_t* max_chunk, int32_t* cluster_size)
{
    std::vector<kap::WorkItem> items;
    std::vector<kap::MergeGroup> groups;
    int32_t mc = 0, rt = 1, cl = 1;
    int32_t slots[kap::kMaxCluster];
    for (int i = 0; i < kap::kMaxCluster; ++i) slots[i] = (i + 1) <= std::max(max_cluster, 1) ? cta_slots / (i + 1) : 0;
    kap_status st = kap::build_schedule(batch, list_len, n_q, num_q_heads, num_kv_heads, slots, slots,
                                        max_chunk_pages, max_items, kap::kRowTile * kap::kMaxRowTiles,
                                        items, groups, &mc, &rt, &cl);
    if (st != KAP_OK) return st;
    if ((int64_t)items.size() > max_items)
        return kap::fail(KAP_ERR_CAPACITY, "%zu items > max_items %d", items.size(), max_items);
    if (items_out && !items.empty())
        std::memcpy(items_out, items.data(), sizeof(kap::WorkItem) * items.size());
    if (n_items) *n_items = (int32_t)items.size();
    if (n_merge_groups) {
        int32_t n = 0;
        for (const auto& g : groups) n += g.n_splits > 1;
        *n_merge_groups = n;
    }
    if (max_chunk) *max_chunk = mc;
    if (cluster_size) *cluster_size = cl;
    return KAP_OK;
}
