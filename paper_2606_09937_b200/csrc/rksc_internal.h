// Internal structures shared by the host-side plan and the kernels.
#pragma once

#include <cstddef>
#include <cstdint>
#include <vector>

#include "rksc.h"

namespace rksc {

constexpr int kBlock = RKSC_BLOCK_SIZE;     // tokens per KV page
constexpr int kMaxRowsPerItem = 64;         // stacked query rows one warp-MMA work item handles
constexpr int kTcMinRows = 9;               // from this many stacked rows on, the tcgen05 kernel takes the item (up to 8: the warp kernel's transposed small-row path)
constexpr int kTcMaxRows = 128;             // rows of one tcgen05 work item (the MMA's M)
constexpr int kMaxPagesPerItem = 512;       // page ids a CTA caches in shared memory
constexpr int kConsumerWarps = 4;           // MMA warps of the segment kernel
constexpr int kWarpKernelThreads = (kConsumerWarps + 2) * 32;   // + two TMA producer warps (K, V)
constexpr int kSubPages = 4;                // pages staged per ring slot
constexpr int kRingSlots = 3;               // ring slots per CTA
constexpr int kCtasPerSm = 2;               // persistent CTAs per SM

// One CTA's work: a chunk of one segment's pages for one KV head and a block of the
// segment's sharers.  Stacked rows = num_sharers * G, row r <-> (sharer r / G, head r % G).
// The plan's item array holds one entry per (chunk, sharer block) with kv_head = 0; work item i is
// entry i / Hkv under KV head h = i % Hkv, its partial rows h * num_sharers * G after the entry's
// (work_item_of below): the Hkv items of a chunk differ in nothing else.
struct WorkItem {
    int32_t seg;
    int32_t kv_head;
    int32_t page_begin;      // absolute index into the flattened page-id array
    int32_t num_pages;
    int32_t num_tokens;      // valid tokens in this chunk
    int32_t sharer_begin;    // absolute index into the sharer array
    int32_t num_sharers;
    int32_t part_row_base;   // first row of this item's partial results
    int32_t seg_page_begin;  // index of the first page within its segment
    int32_t klass;           // 0: warp-MMA kernel, 1: tcgen05 kernel
};
static_assert(sizeof(WorkItem) == 40, "WorkItem is read as 10 int32");

// Work item i of a plan whose item array is `entries` (host and device).
#ifdef __CUDACC__
__host__ __device__
#endif
inline WorkItem work_item_of(const WorkItem* entries, int i, int Hkv, int G) {
    const int e = i / Hkv, h = i - e * Hkv;
    WorkItem w = entries[e];
    w.kv_head = h;
    w.part_row_base += h * w.num_sharers * G;
    return w;
}

// A (segment, branch) incidence: where the branch's masses of this segment start.
struct Sharer {
    int32_t branch;
    int32_t nblk;            // logical blocks of the branch = stride between heads in block_mass
    int64_t mass_base;       // mass_off[branch] * Hq + logical block offset of the segment
};

struct DevicePlan {
    const WorkItem* items = nullptr;
    const int32_t* seg_blocks = nullptr;
    const Sharer* sharers = nullptr;
    const int32_t* merge_off = nullptr;   // [B*Hkv + 1]
    const int32_t* merge_rows = nullptr;  // partial row of head-in-group 0 for each part
    const int64_t* mass_off = nullptr;    // [B+1]
    const int32_t* br_nblk = nullptr;     // [B]
    const int32_t* seg_block_off = nullptr;   // [S+1]
    const int32_t* seg_sharer_off = nullptr;  // [S+1]
    const int32_t* score_chunks = nullptr;    // (segment, first page) pairs, 32 pages each: the score kernel's grid
    int32_t* counters = nullptr;          // [4] work-claim counters (warp kernel, tcgen05 kernel), zero between launches
};

struct HostPlan {
    rksc_layout layout{};
    int32_t B = 0, S = 0, G = 1;
    std::vector<int32_t> seg_blocks;      // flattened page ids of all segments
    std::vector<int32_t> seg_block_off;
    std::vector<int32_t> seg_num_tokens;
    std::vector<WorkItem> items;
    int32_t num_work_items = 0;           // items.size() * Hkv
    int32_t num_tc_items = 0;             // work items [0, num_tc_items) belong to the tcgen05 kernel
    int32_t grid_tc = 0, grid_warp = 0;   // persistent CTAs of the two segment kernels
    std::vector<Sharer> sharers;
    std::vector<int32_t> seg_sharer_off;  // [S+1]
    std::vector<int32_t> merge_off;
    std::vector<int32_t> merge_rows;
    std::vector<int32_t> score_chunks;    // (segment, first page) pairs of the page-score kernel
    std::vector<int64_t> mass_off;        // [B+1]
    std::vector<int32_t> br_nblk;         // [B]
    int64_t mass_elems = 0;
    int32_t num_partial_rows = 0;
    int64_t unique_kv_tokens = 0, duplicated_kv_tokens = 0;
    size_t workspace_bytes = 0;
    size_t ws_lse_offset = 0;             // byte offset of the lse array inside the workspace
    // scratch of build_host_plan, kept so that a recycled plan object allocates nothing
    std::vector<WorkItem> scratch_items;
    std::vector<int32_t> scratch_a, scratch_b;

    // Back to an empty plan; the vectors keep their capacity.
    void reset() {
        layout = rksc_layout{};
        B = S = 0;
        G = 1;
        seg_blocks.clear();
        seg_block_off.clear();
        seg_num_tokens.clear();
        items.clear();
        num_work_items = num_tc_items = grid_tc = grid_warp = 0;
        sharers.clear();
        seg_sharer_off.clear();
        merge_off.clear();
        merge_rows.clear();
        score_chunks.clear();
        mass_off.clear();
        br_nblk.clear();
        mass_elems = 0;
        num_partial_rows = 0;
        unique_kv_tokens = duplicated_kv_tokens = 0;
        workspace_bytes = ws_lse_offset = 0;
    }
};

// Builds every host list from validated tables.  num_sms sizes the KV chunks.
int32_t build_host_plan(const rksc_layout& layout, const rksc_tables& t, int num_sms, HostPlan* hp);

}  // namespace rksc

namespace rksc {
// Device memory of a plan's lists, with the pinned buffer they are staged in; recycled between plans.
struct PlanArena {
    void* dev = nullptr;
    void* host = nullptr;          // pinned
    size_t capacity = 0;
    int device = -1;
    struct CUevent_st* done = nullptr;   // cudaEvent_t, recorded when a plan that ran is destroyed
    bool busy = false;
};
}  // namespace rksc

struct rksc_plan {
    rksc::HostPlan host;
    rksc::DevicePlan dev;
    rksc::PlanArena arena;
    mutable bool used = false;          // a launch was enqueued with this plan
    mutable void* last_stream = nullptr;
    int device = -1;
    int num_sms = 148;
    bool on_device = false;
};
