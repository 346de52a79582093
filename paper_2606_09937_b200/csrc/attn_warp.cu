// Segment attention with warp-level MMA (stacked rows <= 64): persistent, warp-specialised.
//
// A work item is a chunk of one segment's KV pages for one KV head plus a block of the branches
// that share the segment.  The query rows of all those branches x the G query heads of the KV
// head are stacked into 16-row tiles, so a page staged in shared memory once serves every
// sharing branch (this is what replaces the paper's B physical copies of the prefix cache,
// Algorithm 1 line 3 / Section 2.2).
//
//   * Persistent CTAs (two per SM) take work items, longest first, from a global counter.
//   * Warp 4 is the producer: it claims items and streams their pages, four pages (K and V,
//     16 tokens each) per ring slot, by TMA (cp.async.bulk.tensor, 128-byte swizzle, 16 x 64
//     boxes) with one mbarrier per slot for arrival and one for release, plus a small header
//     per slot (item, position, last-slot flag) that the consumers follow.  It runs ahead
//     across item boundaries, so the ring never drains between items.  No cluster multicast.
//   * Warps 0-3 are consumers.  With R stacked rows there are nrt = ceil(R/16) row tiles; the
//     warps are arranged as (row tile) x (page lane): PL = 4, 2 or 1 page lanes split the pages of
//     every slot among them, and the row-tile warps of a lane read the same staged page.
//   * Per page and warp: S = Q K^T by mma.sync m16n8k16 (bf16 in, fp32 out), online softmax in
//     base 2, P split into a bf16 high and low part (two MMAs) so that P V carries fp32-level
//     error, and the page's softmax mass written as log2 (absolute, independent of the running
//     maximum) for the merge kernel to normalise.  The accumulator is rescaled only on pages
//     where a running maximum moved.
//   * Items with at most 8 stacked rows (a private suffix or prefix copy: R = G) use the
//     transposed product S^T = K Q^T (M = 16 tokens, N = 8 rows), O^T = V^T P^T: no padding of
//     the rows to 16, half the MMAs, a quarter of the softmax work per thread; P^T reaches the
//     B-operand layout with movmatrix.
//   * At the end of an item the page lanes are merged through a small shared-memory scratch
//     (32 columns at a time) and the item's partial (normalised O, log2-sum-exp) goes to the
//     workspace.
// Every mbarrier wait is bounded; on expiry the CTA records RKSC_ERR_DEVICE_TIMEOUT, stops
// issuing copies, skips further waits and runs to completion.
#include <cuda_bf16.h>

#include "kernels.h"

namespace rksc {

namespace {

constexpr int kThreads = kWarpKernelThreads;
constexpr int kCW = kConsumerWarps;
constexpr int kNS = kRingSlots;
constexpr int kSP = kSubPages;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive_n(uint32_t bar, uint32_t n) {   // n arrivals at once
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(n) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after 2^32 SM cycles (about two seconds).  The SM cycle counter is a
// cheap register read, so polling it costs nothing next to the barrier probe itself.
// With a suspend-time hint (nanoseconds) the thread sleeps in hardware until the phase completes
// or the time is up, instead of polling and taking issue slots from the working warps.
__device__ __forceinline__ bool mbar_try_wait_sleep(uint32_t bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity), "r"(ns)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_test(uint32_t bar, uint32_t parity) {   // never blocks
    uint32_t ok;
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n"
        "selp.u32 %0, 1, 0, p;\n"
        "}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait_sleep(bar, parity, 20000u)) return true;
        if (clock64() - t0 > (1ll << 32)) return false;
    }
}
// Keys and values are read once per launch: their lines are marked first to leave L2, so that the
// partial results and block masses written meanwhile are still there when the merge reads them.
__device__ __forceinline__ uint64_t l2_evict_first_policy() {
    uint64_t pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ float fast_log2(float x) {
    float y;
    asm volatile("lg2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// p -> bf16 high part and bf16 residual, two values packed per register (lower index low)
__device__ __forceinline__ void split_pack(float a, float b, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(a - hf.x, b - hf.y);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
}

#ifdef RKSC_WAIT_PROFILE
// Development aid: per-CTA cycle counts of where the producer and consumer warp 0 wait.
// [cta][0] total, [1] producer waits for a free slot, [2] consumer waits for data,
// [3] consumer item set-up, [4] consumer epilogue, [5] items, [6] slots.
__device__ unsigned long long g_wait_prof[1024][8];
#define PROF_T0() const long long _t0 = clock64()
#define PROF_ADD(i) if (lane == 0) g_wait_prof[blockIdx.x][i] += (unsigned long long)(clock64() - _t0)
#define PROF_INC(i) if (lane == 0) g_wait_prof[blockIdx.x][i] += 1ull
#else
#define PROF_T0()
#define PROF_ADD(i)
#define PROF_INC(i)
#endif

// What the producer tells the consumers about a ring slot.
struct __align__(16) SlotHeader {
    int32_t item;        // index of the work item, -1: no more work
    int32_t group;       // position of this slot within the item (0 = first)
    int32_t num_pages;   // pages staged in this slot (1..kSP)
    int32_t last;        // 1 on the item's last slot
    WorkItem it;         // the item itself, so that consumers need not fetch it
    int32_t pad[2];
};
static_assert(sizeof(SlotHeader) == 64, "SlotHeader is written as four 16-byte stores");

template <int HD>
struct SmemLayout {
    static constexpr int kTile = kBlock * HD * 2;          // bytes of one K (or V) page tile
    static constexpr int kPage = 2 * kTile;                // K then V of one page
    static constexpr int kSlot = kSP * kPage;
    static constexpr int kRing = kNS * kSlot;
    static constexpr int kScrRow = 40;                     // floats per scratch row (32 columns + pad)
    static constexpr int kScrWarp = 16 * kScrRow * 4;      // bytes per warp
    static constexpr int kScrOff = kRing;
    static constexpr int kMlOff = kScrOff + kCW * kScrWarp;   // m[4][16], l[4][16]
    static constexpr int kBarOff = kMlOff + 2 * kCW * 16 * 4;  // full[kNS], empty[kNS]
    static constexpr int kHdrOff = kBarOff + ((4 * kNS * 8 + 8 + 15) / 16) * 16;  // after the barriers: full, empty, consumers' own, header ready, partials ready
    static_assert(kBarOff % 8 == 0 && kHdrOff % 16 == 0 && kScrOff % 16 == 0, "shared-memory alignment");
    static constexpr int kPagesOff = kHdrOff + kNS * 64;       // one SlotHeader per slot, then its page ids
    static constexpr int kFlagOff = kPagesOff + kNS * kSP * 4;
    // an item with <= 8 rows merges its four page lanes through the sub-page regions of its last slot
    static_assert(8 * (HD + 4) * 4 + 64 <= kPage, "small-row merge scratch must fit in a sub-page");
    static constexpr int kTotal = kFlagOff + 16;
};

template <int HD>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
seg_attn_warp_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                     const AttnArgs a) {
    using SL = SmemLayout<HD>;
    constexpr int KS = HD / 16;      // k-steps of Q K^T (and 16-wide tiles of d)
    constexpr int NT = HD / 8;       // n-tiles of P V
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t ring = smem_u32(smem);
    const uint32_t bar_full = ring + SL::kBarOff;
    const uint32_t bar_empty = bar_full + kNS * 8;
    const uint32_t bar_cons = bar_empty + kNS * 8;   // the four consumer warps meet here in the item epilogue
    const uint32_t bar_hdr = bar_cons + 8;           // [kNS] header and page ids of the slot written (K producer -> V producer)
    const uint32_t bar_epi = bar_hdr + kNS * 8;      // [kNS] a small-row item's page-lane states are in this slot's memory (consumers -> V producer)
    SlotHeader* s_hdr = reinterpret_cast<SlotHeader*>(smem + SL::kHdrOff);
    int32_t* s_pages = reinterpret_cast<int32_t*>(smem + SL::kPagesOff);
    volatile int32_t* s_abort = reinterpret_cast<volatile int32_t*>(smem + SL::kFlagOff);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < kNS; ++i) {
            mbar_init(bar_full + 8 * i, 2);     // the K and the V producer
            mbar_init(bar_empty + 8 * i, kCW);
            mbar_init(bar_hdr + 8 * i, 1);
            mbar_init(bar_epi + 8 * i, kCW);
        }
        mbar_init(bar_cons, kCW);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // the merge kernel may be made resident early; it waits for this grid's completion itself
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    __syncthreads();

    auto wait_or_abort = [&](uint32_t bar, uint32_t parity) {
        if (*s_abort) return;
        if (!mbar_wait(bar, parity)) {
            *s_abort = 1;
            if (a.status) atomicExch(a.status, RKSC_ERR_DEVICE_TIMEOUT);
        }
    };

    if (warp == kCW) {
        // ------------------------------ producer warp ------------------------------
        // Two claimed items are kept ahead of the one being streamed, and page ids are fetched 32
        // at a time one batch ahead, so that no global-memory latency sits between two TMA issues.
        auto claim = [&]() {   // this kernel's items follow the tcgen05 kernel's in the item array
            int v = 0;
            if (lane == 0) v = a.num_tc_items + atomicAdd(a.counters, 1);
            return __shfl_sync(0xffffffffu, v, 0);
        };
        auto fetch_item = [&](int i) {
            WorkItem w{};
            if (i < a.num_items) w = work_item_of(a.plan.items, i, a.Hkv, a.G);
            return w;
        };
        auto fetch_ids = [&](const WorkItem& w, int first) {   // page ids first + lane of the item (0 past its end)
            return (first + lane < w.num_pages) ? __ldg(a.plan.seg_blocks + w.page_begin + first + lane) : 0;
        };
        const uint64_t kv_policy = l2_evict_first_policy();
        int seq = 0;
        int idx = claim();
        WorkItem it = fetch_item(idx);
        int ids = fetch_ids(it, 0);
        int nidx = claim();
        WorkItem nit = fetch_item(nidx);
        int nids = fetch_ids(nit, 0);
        while (idx < a.num_items && !*s_abort) {
            const int nnidx = claim();   // two items ahead: its latency hides behind this whole item
            const int ngroups = (it.num_pages + kSP - 1) / kSP;
            int ids_ahead = 0;
            for (int g = 0; g < ngroups; ++g, ++seq) {
                const int slot = seq % kNS;
                const int npg = min(kSP, it.num_pages - g * kSP);
                if ((g & 7) == 0) ids_ahead = fetch_ids(it, (g + 8) * kSP);   // the batch after this one
                const int page = __shfl_sync(0xffffffffu, ids, (g & 7) * kSP + (lane & (kSP - 1)));
                if ((g & 7) == 7) ids = ids_ahead;
                {
                    PROF_T0();
                    if (seq >= kNS) wait_or_abort(bar_empty + 8 * slot, (uint32_t)(seq / kNS - 1) & 1u);
                    PROF_ADD(1);
                }
                if (*s_abort) break;
                const uint32_t bar = bar_full + 8 * slot;
                if (lane == 0) {
                    SlotHeader h;
                    h.item = idx;
                    h.group = g;
                    h.num_pages = npg;
                    h.last = (g == ngroups - 1);
                    h.it = it;
                    h.pad[0] = h.pad[1] = 0;
                    s_hdr[slot] = h;
                }
                if (lane < kSP) s_pages[slot * kSP + lane] = page;
                __syncwarp();
                if (lane == 0) {
                    mbar_arrive(bar_hdr + 8 * slot);                 // the V producer may follow
                    mbar_arrive_expect_tx(bar, npg * SL::kTile);     // this warp's half of the slot: K
                }
                __syncwarp();
                if (lane < npg) {
                    const int y = (page * a.Hkv + it.kv_head) * kBlock;
                    const uint32_t dst = ring + slot * SL::kSlot + lane * SL::kPage;
#pragma unroll
                    for (int hh = 0; hh < HD / 64; ++hh) tma_load_2d(dst + hh * 2048, &tm_k, hh * 64, y, bar, kv_policy);
                }
            }
            idx = nidx;
            it = nit;
            ids = nids;
            nidx = nnidx;
            nit = fetch_item(nidx);
            nids = fetch_ids(nit, 0);
        }
        // end marker for the consumers
        {
            const int slot = seq % kNS;
            if (seq >= kNS) wait_or_abort(bar_empty + 8 * slot, (uint32_t)(seq / kNS - 1) & 1u);
            if (lane == 0) {
                s_hdr[slot].item = -1;
                mbar_arrive(bar_hdr + 8 * slot);
                mbar_arrive(bar_full + 8 * slot);
            }
        }
        // the last CTA to stop claiming items rewinds the counters for the next launch
        if (lane == 0) {
            __threadfence();
            const int done = atomicAdd(a.counters + 1, 1);
            if (done == (int)gridDim.x - 1) {
                a.counters[0] = 0;
                a.counters[1] = 0;
                __threadfence();
            }
        }
        // When this grid was launched behind the tcgen05 kernel without waiting for it, it must not
        // complete before that kernel has: the merge kernel waits on this grid only.
        asm volatile("griddepcontrol.wait;" ::: "memory");
        return;
    }

    if (warp == kCW + 1) {
        // ------------------------------ V producer warp ------------------------------
        // One warp cannot issue TMA copies fast enough for a CTA's share of the memory bandwidth: this
        // one follows the K producer slot by slot (header and page ids through shared memory) and
        // issues the V half of every slot.
        // It also finishes the small-row items (<= 8 stacked rows: the four consumer warps were four page
        // lanes of the same rows): the consumers leave their lane states in the memory of the item's
        // last slot, signal bar_epi and go on to the next item; this warp, which waits most of the
        // time, merges the lanes, writes the partial result and releases the slot.
        const uint64_t kv_policy = l2_evict_first_policy();
        uint32_t pending = 0;    // ring slots that hold such lane states (or will, once the consumers get there)
        uint32_t epi_par = 0;    // per ring slot: parity of its next bar_epi phase
        auto finish_item = [&](int slot) {
            constexpr int RS = HD + 4, CPL = HD / 32;   // row stride of a lane's O^T, columns per thread here
            const WorkItem w = s_hdr[slot].it;
            const int nrows = w.num_sharers * a.G;
            const size_t prow0 = (size_t)w.part_row_base;
            const float* base = reinterpret_cast<const float*>(smem + slot * SL::kSlot);
            for (int row = 0; row < nrows; ++row) {
                float mw[kCW], M = -INFINITY;
#pragma unroll
                for (int p = 0; p < kCW; ++p) {
                    mw[p] = base[p * (SL::kPage / 4) + 8 * RS + row];
                    M = fmaxf(M, mw[p]);
                }
                float lsum = 0.f, acc[CPL];
#pragma unroll
                for (int c = 0; c < CPL; ++c) acc[c] = 0.f;
#pragma unroll
                for (int p = 0; p < kCW; ++p) {
                    const float* wl = base + p * (SL::kPage / 4);
                    const float wt = (mw[p] == -INFINITY) ? 0.f : fast_exp2(mw[p] - M);
                    lsum += wt * wl[8 * RS + 8 + row];
#pragma unroll
                    for (int c = 0; c < CPL; ++c) acc[c] += wt * wl[row * RS + CPL * lane + c];
                }
                float* dst = a.part_o + (prow0 + row) * HD + CPL * lane;
#pragma unroll
                for (int c = 0; c < CPL; ++c) dst[c] = acc[c] / lsum;
                if (lane == 0) a.part_lse[prow0 + row] = M + fast_log2(lsum);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive_n(bar_empty + 8 * slot, kCW);   // in the consumers' stead
            pending &= ~(1u << slot);
            epi_par ^= 1u << slot;
        };
        for (int seq = 0; !*s_abort; ++seq) {
            const int slot = seq % kNS;
            // The K producer cannot publish this ring slot again before the item that ended in it is
            // finished: do that first.  The other slots are looked at in passing.
#pragma unroll
            for (int s2 = 0; s2 < kNS; ++s2) {
                if (!(pending & (1u << s2))) continue;
                const uint32_t par = (epi_par >> s2) & 1u;
                if (s2 == slot) {
                    wait_or_abort(bar_epi + 8 * s2, par);
                    if (*s_abort) break;
                    finish_item(s2);
                } else if (__all_sync(0xffffffffu, mbar_test(bar_epi + 8 * s2, par))) {
                    finish_item(s2);
                }
            }
            if (*s_abort) break;
            wait_or_abort(bar_hdr + 8 * slot, (uint32_t)(seq / kNS) & 1u);
            if (*s_abort) break;
            const int item = s_hdr[slot].item;
            const uint32_t bar = bar_full + 8 * slot;
            if (item < 0) {
                if (lane == 0) mbar_arrive(bar);
                // the items still to be finished
#pragma unroll
                for (int s2 = 0; s2 < kNS; ++s2) {
                    if (!(pending & (1u << s2)) || *s_abort) continue;
                    wait_or_abort(bar_epi + 8 * s2, (epi_par >> s2) & 1u);
                    if (!*s_abort) finish_item(s2);
                }
                break;
            }
            const int npg = s_hdr[slot].num_pages;
            const int kvh = s_hdr[slot].it.kv_head;
            const bool ends_small = s_hdr[slot].last && s_hdr[slot].it.num_sharers * a.G <= 8;
            const int page = s_pages[slot * kSP + (lane & (kSP - 1))];
            __syncwarp();
            if (lane == 0) mbar_arrive_expect_tx(bar, npg * SL::kTile);
            __syncwarp();
            if (lane < npg) {
                const int y = (page * a.Hkv + kvh) * kBlock;
                const uint32_t dst = ring + slot * SL::kSlot + lane * SL::kPage + SL::kTile;
#pragma unroll
                for (int hh = 0; hh < HD / 64; ++hh) tma_load_2d(dst + hh * 2048, &tm_v, hh * 64, y, bar, kv_policy);
            }
            if (ends_small) pending |= 1u << slot;
        }
        return;
    }

    // -------------------------------- consumer warps --------------------------------
    const int g4 = lane >> 2, t = lane & 3;
    // per-lane ldmatrix row/chunk selectors (two mappings; each path uses one per operand)
    const int a_tok = ((lane >> 4) << 3) + (lane & 7);       // matrices ordered (tok lo, +chunk), (tok hi, ...)
    const int a_chunk = (lane >> 3) & 1;
    const int b_tok = (((lane >> 3) & 1) << 3) + (lane & 7); // matrices ordered (tok lo), (tok hi), then +chunk
    const int b_chunk = lane >> 4;
    const uint32_t a_lane_off = a_tok * 128, b_lane_off = b_tok * 128;
    const float scale_log2 = a.scale_log2;
    const int G = a.G;
    float* scr = reinterpret_cast<float*>(smem + SL::kScrOff);
    float* s_m = reinterpret_cast<float*>(smem + SL::kMlOff);
    float* s_l = s_m + kCW * 16;
    uint32_t cons_phase = 0;
    // Bounded meeting of the consumer warps (shared-memory writes before it are visible after it).
    auto consumer_sync = [&]() {
#ifdef RKSC_EPI_BARSYNC
        asm volatile("bar.sync 1, 128;" ::: "memory");
#else
        __syncwarp();
        if (lane == 0) mbar_arrive(bar_cons);
        wait_or_abort(bar_cons, cons_phase);
        cons_phase ^= 1u;
#endif
    };

    // item state
    WorkItem it{};
    int rows = 0, nrt = 1, nrtp = 1, PL = kCW, rt = 0, pl = warp;
    bool active = false, small_rows = false, v0 = false, v1 = false;
    int r0 = 0, r1 = 0;            // the two stacked rows this thread owns in the softmax
    int64_t mb0 = 0, mb1 = 0;      // their positions in block_mass
    uint32_t qf[KS][4];
    float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
    float o[NT][4];

#ifdef RKSC_WAIT_PROFILE
    const long long t_begin = clock64();
#endif
    for (int seq = 0;; ++seq) {
        const int slot = seq % kNS;
        {
            PROF_T0();
            wait_or_abort(bar_full + 8 * slot, (uint32_t)(seq / kNS) & 1u);
            if (warp == 0) { PROF_ADD(2); PROF_INC(6); }
        }
        const int4 hdr = *reinterpret_cast<const int4*>(&s_hdr[slot]);   // item, group, pages, last
#ifdef RKSC_WAIT_PROFILE
        if (hdr.x < 0 && warp == 0 && lane == 0) g_wait_prof[blockIdx.x][0] += (unsigned long long)(clock64() - t_begin);
        const long long t_item = clock64();
#endif
        if (hdr.x < 0 || *s_abort) break;
        const int g = hdr.y, npg = hdr.z;

        if (g == 0) {
            // ---- new item: rows, queries, running state ----
            it = s_hdr[slot].it;
            rows = it.num_sharers * G;
            small_rows = rows <= 8;
            nrt = (rows + 15) >> 4;
            nrtp = (nrt == 3) ? 4 : nrt;
            PL = kCW / nrtp;
            rt = warp % nrtp;
            pl = warp / nrtp;
            active = rt < nrt;
            // general path: thread rows rt*16 + g4 (+8), queries of the same rows (A operand);
            // small path: thread rows 2t, 2t+1, query of row g4 (B operand)
            r0 = small_rows ? 2 * t : rt * 16 + g4;
            r1 = small_rows ? 2 * t + 1 : r0 + 8;
            v0 = active && r0 < rows;
            v1 = active && r1 < rows;
            const int qr0 = small_rows ? g4 : r0, qr1 = r1;
            const bool qv0 = active && qr0 < rows, qv1 = !small_rows && v1;
            const uint32_t* q0 = nullptr;
            const uint32_t* q1 = nullptr;
            if (v0) {
                const Sharer sh = a.plan.sharers[it.sharer_begin + r0 / G];
                const int h = it.kv_head * G + r0 % G;
                mb0 = sh.mass_base + (int64_t)h * sh.nblk + it.seg_page_begin;
            }
            if (v1) {
                const Sharer sh = a.plan.sharers[it.sharer_begin + r1 / G];
                const int h = it.kv_head * G + r1 % G;
                mb1 = sh.mass_base + (int64_t)h * sh.nblk + it.seg_page_begin;
            }
            if (qv0) {
                const int br = a.plan.sharers[it.sharer_begin + qr0 / G].branch;
                q0 = reinterpret_cast<const uint32_t*>(a.q) + ((size_t)br * a.Hq + it.kv_head * G + qr0 % G) * (HD / 2);
            }
            if (qv1) {
                const int br = a.plan.sharers[it.sharer_begin + qr1 / G].branch;
                q1 = reinterpret_cast<const uint32_t*>(a.q) + ((size_t)br * a.Hq + it.kv_head * G + qr1 % G) * (HD / 2);
            }
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qf[ks][0] = qv0 ? __ldg(q0 + ks * 8 + t) : 0u;
                qf[ks][2] = qv0 ? __ldg(q0 + ks * 8 + 4 + t) : 0u;
                qf[ks][1] = qv1 ? __ldg(q1 + ks * 8 + t) : 0u;
                qf[ks][3] = qv1 ? __ldg(q1 + ks * 8 + 4 + t) : 0u;
            }
            m0 = m1 = -INFINITY;
            l0 = l1 = 0.f;
#pragma unroll
            for (int n = 0; n < NT; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;
#ifdef RKSC_WAIT_PROFILE
            if (warp == 0 && lane == 0) {
                g_wait_prof[blockIdx.x][3] += (unsigned long long)(clock64() - t_item) + (qf[0][0] & 1u) * 0ull;
                g_wait_prof[blockIdx.x][5] += 1ull;
            }
#endif
        }

#ifdef RKSC_WAIT_PROFILE
        const long long t_pages = clock64();
#endif
#ifdef RKSC_SKIP_COMPUTE
        if (false) {
#else
        if (active) {
#endif
            for (int j = pl; j < npg; j += PL) {
                const uint32_t kb = ring + slot * SL::kSlot + j * SL::kPage;
                const uint32_t vb = kb + SL::kTile;
                const int pi = g * kSP + j;                   // page index within the item
                const int nv = it.num_tokens - pi * kBlock;   // valid tokens: >= 1, >= 16 if full

                if (small_rows) {
                    // ---- S^T = K Q^T: 16 tokens x 8 rows; thread: tokens g4, g4+8; rows 2t, 2t+1 ----
                    float s[4] = {0.f, 0.f, 0.f, 0.f}, s_odd[4] = {0.f, 0.f, 0.f, 0.f};   // two chains over d
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int chunk = ((ks * 2) & 7) + b_chunk;
                        const uint32_t addr = kb + (ks >> 2) * 2048 + b_lane_off + ((chunk ^ (b_tok & 7)) << 4);
                        uint32_t ak[4];
                        ldmatrix_x4(addr, ak);
                        if (ks & 1) mma_bf16(s_odd, ak, qf[ks][0], qf[ks][2]);
                        else mma_bf16(s, ak, qf[ks][0], qf[ks][2]);
                    }
#pragma unroll
                    for (int e = 0; e < 4; ++e) s[e] += s_odd[e];
                    s[0] = (g4 < nv) ? s[0] * scale_log2 : -INFINITY;
                    s[1] = (g4 < nv) ? s[1] * scale_log2 : -INFINITY;
                    s[2] = (g4 + 8 < nv) ? s[2] * scale_log2 : -INFINITY;
                    s[3] = (g4 + 8 < nv) ? s[3] * scale_log2 : -INFINITY;
                    float mx0 = fmaxf(s[0], s[2]), mx1 = fmaxf(s[1], s[3]);
#pragma unroll
                    for (int sh = 4; sh <= 16; sh <<= 1) {
                        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, sh));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, sh));
                    }
                    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                    const bool moved = (mn0 != m0) || (mn1 != m1);
                    const float al0 = fast_exp2(m0 - mn0), al1 = fast_exp2(m1 - mn1);
                    m0 = mn0;
                    m1 = mn1;
                    float p[4];
                    p[0] = fast_exp2(s[0] - mn0);
                    p[1] = fast_exp2(s[1] - mn1);
                    p[2] = fast_exp2(s[2] - mn0);
                    p[3] = fast_exp2(s[3] - mn1);
                    float rs0 = p[0] + p[2], rs1 = p[1] + p[3];
#pragma unroll
                    for (int sh = 4; sh <= 16; sh <<= 1) {
                        rs0 += __shfl_xor_sync(0xffffffffu, rs0, sh);
                        rs1 += __shfl_xor_sync(0xffffffffu, rs1, sh);
                    }
                    l0 = l0 * al0 + rs0;
                    l1 = l1 * al1 + rs1;
                    if (a.block_mass != nullptr && g4 == 0) {
                        if (v0) a.block_mass[mb0 + pi] = mn0 + fast_log2(rs0);
                        if (v1) a.block_mass[mb1 + pi] = mn1 + fast_log2(rs1);
                    }
                    if (__any_sync(0xffffffffu, moved)) {
#pragma unroll
                        for (int n = 0; n < 2 * KS; ++n) {
                            o[n][0] *= al0;
                            o[n][1] *= al1;
                            o[n][2] *= al0;
                            o[n][3] *= al1;
                        }
                    }
                    // P^T (tokens x rows) -> B operand (k = token pairs, n = row) by 8x8 transposes
                    uint32_t h01, l01, h23, l23;
                    split_pack(p[0], p[1], h01, l01);
                    split_pack(p[2], p[3], h23, l23);
                    const uint32_t bh0 = movmatrix_trans(h01), bh1 = movmatrix_trans(h23);
                    const uint32_t bl0 = movmatrix_trans(l01), bl1 = movmatrix_trans(l23);
                    // O^T += V^T P^T: 16 values of d per tile
#pragma unroll
                    for (int n = 0; n < KS; ++n) {
                        const int chunk = ((n * 2) & 7) + a_chunk;
                        const uint32_t addr = vb + (n >> 2) * 2048 + a_lane_off + ((chunk ^ (a_tok & 7)) << 4);
                        uint32_t av[4];
                        ldmatrix_x4_trans(addr, av);
                        mma_bf16(o[n], av, bh0, bh1);          // high parts of P accumulate in o[0..KS)
                        mma_bf16(o[KS + n], av, bl0, bl1);     // low parts in o[KS..2KS): no dependent pair
                    }
                } else {
                    // ---- S = Q K^T for 16 rows x 16 tokens ----
                    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int chunk = ((ks * 2) & 7) + a_chunk;
                        const uint32_t addr = kb + (ks >> 2) * 2048 + a_lane_off + ((chunk ^ (a_tok & 7)) << 4);
                        uint32_t bk[4];
                        ldmatrix_x4(addr, bk);
                        mma_bf16(s[0], qf[ks], bk[0], bk[1]);
                        mma_bf16(s[1], qf[ks], bk[2], bk[3]);
                    }
                    // mask the tail of a partial page, move to log2 units
#pragma unroll
                    for (int n = 0; n < 2; ++n)
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const int tok = n * 8 + 2 * t + (e & 1);
                            s[n][e] = (tok < nv) ? s[n][e] * scale_log2 : -INFINITY;
                        }
                    float mx0 = fmaxf(fmaxf(s[0][0], s[0][1]), fmaxf(s[1][0], s[1][1]));
                    float mx1 = fmaxf(fmaxf(s[0][2], s[0][3]), fmaxf(s[1][2], s[1][3]));
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 1));
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, 2));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 1));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, 2));
                    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                    const bool moved = (mn0 != m0) || (mn1 != m1);
                    const float al0 = fast_exp2(m0 - mn0), al1 = fast_exp2(m1 - mn1);
                    m0 = mn0;
                    m1 = mn1;
                    float p[2][4];
#pragma unroll
                    for (int n = 0; n < 2; ++n) {
                        p[n][0] = fast_exp2(s[n][0] - mn0);
                        p[n][1] = fast_exp2(s[n][1] - mn0);
                        p[n][2] = fast_exp2(s[n][2] - mn1);
                        p[n][3] = fast_exp2(s[n][3] - mn1);
                    }
                    float rs0 = (p[0][0] + p[0][1]) + (p[1][0] + p[1][1]);
                    float rs1 = (p[0][2] + p[0][3]) + (p[1][2] + p[1][3]);
                    rs0 += __shfl_xor_sync(0xffffffffu, rs0, 1);
                    rs0 += __shfl_xor_sync(0xffffffffu, rs0, 2);
                    rs1 += __shfl_xor_sync(0xffffffffu, rs1, 1);
                    rs1 += __shfl_xor_sync(0xffffffffu, rs1, 2);
                    l0 = l0 * al0 + rs0;
                    l1 = l1 * al1 + rs1;
                    if (a.block_mass != nullptr && t == 0) {
                        // log2 of the page's unnormalised mass, absolute (not relative to the running max)
                        if (v0) a.block_mass[mb0 + pi] = mn0 + fast_log2(rs0);
                        if (v1) a.block_mass[mb1 + pi] = mn1 + fast_log2(rs1);
                    }
                    if (__any_sync(0xffffffffu, moved)) {
#pragma unroll
                        for (int n = 0; n < NT; ++n) {
                            o[n][0] *= al0;
                            o[n][1] *= al0;
                            o[n][2] *= al1;
                            o[n][3] *= al1;
                        }
                    }
                    // O += P V, P as bf16 high + low parts
                    uint32_t phi[4], plo[4];
                    split_pack(p[0][0], p[0][1], phi[0], plo[0]);
                    split_pack(p[0][2], p[0][3], phi[1], plo[1]);
                    split_pack(p[1][0], p[1][1], phi[2], plo[2]);
                    split_pack(p[1][2], p[1][3], phi[3], plo[3]);
#pragma unroll
                    for (int np = 0; np < NT / 2; ++np) {
                        const int chunk = ((np * 2) & 7) + b_chunk;
                        const uint32_t addr = vb + (np >> 2) * 2048 + b_lane_off + ((chunk ^ (b_tok & 7)) << 4);
                        uint32_t bv[4];
                        ldmatrix_x4_trans(addr, bv);
                        mma_bf16(o[2 * np], phi, bv[0], bv[1]);
                        mma_bf16(o[2 * np], plo, bv[0], bv[1]);
                        mma_bf16(o[2 * np + 1], phi, bv[2], bv[3]);
                        mma_bf16(o[2 * np + 1], plo, bv[2], bv[3]);
                    }
                }
            }
        }
#ifdef RKSC_WAIT_PROFILE
        if (warp == 0 && lane == 0) g_wait_prof[blockIdx.x][7] += (unsigned long long)(clock64() - t_pages) + (__float_as_uint(o[0][0]) & 1u) * 0ull;
#endif
        // release the slot, except on the last slot of a small-row item, whose memory serves the merge
        if (!(hdr.w && small_rows)) {
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
        }
        if (!hdr.w) continue;
        PROF_T0();

        // ---- item epilogue: merge the page lanes, write the partial (normalised O, log2-sum-exp) ----
        const size_t prow0 = (size_t)it.part_row_base;
        if (small_rows) {
            // Warp w was the only reader of sub-page w of this slot, so it may overwrite that region
            // with its partial state right away: [8 rows][HD + 4] floats of O^T, then m[8], l[8].
            constexpr int RS = HD + 4;
            float* base = reinterpret_cast<float*>(smem + slot * SL::kSlot);
            float* mine = base + warp * (SL::kPage / 4);
#pragma unroll
            for (int n = 0; n < KS; ++n) {
                mine[(2 * t) * RS + n * 16 + g4] = o[n][0] + o[KS + n][0];
                mine[(2 * t + 1) * RS + n * 16 + g4] = o[n][1] + o[KS + n][1];
                mine[(2 * t) * RS + n * 16 + g4 + 8] = o[n][2] + o[KS + n][2];
                mine[(2 * t + 1) * RS + n * 16 + g4 + 8] = o[n][3] + o[KS + n][3];
            }
            if (g4 == 0) {
                mine[8 * RS + 2 * t] = m0;
                mine[8 * RS + 2 * t + 1] = m1;
                mine[8 * RS + 8 + 2 * t] = l0;
                mine[8 * RS + 8 + 2 * t + 1] = l1;
            }
            // the V producer warp merges the four lanes, writes the partial and releases the slot
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_epi + 8 * slot);
        } else if (PL == 1) {
            // one warp per row tile: straight from registers
            if (active) {
                const float i0 = 1.f / l0, i1 = 1.f / l1;
                if (v0) {
                    float* dst = a.part_o + (prow0 + r0) * HD + 2 * t;
#pragma unroll
                    for (int n = 0; n < NT; ++n)
                        *reinterpret_cast<float2*>(dst + n * 8) = make_float2(o[n][0] * i0, o[n][1] * i0);
                    if (t == 0) a.part_lse[prow0 + r0] = m0 + fast_log2(l0);
                }
                if (v1) {
                    float* dst = a.part_o + (prow0 + r1) * HD + 2 * t;
#pragma unroll
                    for (int n = 0; n < NT; ++n)
                        *reinterpret_cast<float2*>(dst + n * 8) = make_float2(o[n][2] * i1, o[n][3] * i1);
                    if (t == 0) a.part_lse[prow0 + r1] = m1 + fast_log2(l1);
                }
            }
        } else {
            // two page lanes hold partial states of the same rows (17..32 rows; all four warps are active)
            if (t == 0) {
                s_m[warp * 16 + g4] = m0;
                s_l[warp * 16 + g4] = l0;
                s_m[warp * 16 + g4 + 8] = m1;
                s_l[warp * 16 + g4 + 8] = l1;
            }
            float* my = scr + warp * (16 * SL::kScrRow);
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
#pragma unroll
                for (int n = 0; n < 4; ++n) {
                    *reinterpret_cast<float2*>(my + g4 * SL::kScrRow + n * 8 + 2 * t) =
                        make_float2(o[4 * c + n][0], o[4 * c + n][1]);
                    *reinterpret_cast<float2*>(my + (g4 + 8) * SL::kScrRow + n * 8 + 2 * t) =
                        make_float2(o[4 * c + n][2], o[4 * c + n][3]);
                }
                consumer_sync();
                if (*s_abort) break;
                for (int idx = tid; idx < rows * 32; idx += kCW * 32) {
                    const int row = idx >> 5, col = idx & 31;
                    const int rtile = row >> 4, rr = row & 15;
                    float M = -INFINITY;
                    for (int p = 0; p < PL; ++p) M = fmaxf(M, s_m[(p * nrtp + rtile) * 16 + rr]);
                    float lsum = 0.f, acc = 0.f;
                    for (int p = 0; p < PL; ++p) {
                        const int w = p * nrtp + rtile;
                        const float mw = s_m[w * 16 + rr];
                        const float wt = (mw == -INFINITY) ? 0.f : fast_exp2(mw - M);
                        lsum += wt * s_l[w * 16 + rr];
                        acc += wt * scr[w * (16 * SL::kScrRow) + rr * SL::kScrRow + col];
                    }
                    a.part_o[(prow0 + row) * HD + c * 32 + col] = acc / lsum;
                    if (c == 0 && col == 0) a.part_lse[prow0 + row] = M + fast_log2(lsum);
                }
                consumer_sync();
                if (*s_abort) break;
            }
        }
        if (warp == 0) { PROF_ADD(4); }
    }
}

}  // namespace

#ifdef RKSC_WAIT_PROFILE
extern "C" __attribute__((visibility("default"))) int rksc_debug_wait_profile(unsigned long long* host_out, int reset) {
    if (host_out && cudaMemcpyFromSymbol(host_out, g_wait_prof, sizeof(g_wait_prof)) != cudaSuccess) return -1;
    if (reset) {
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_wait_prof) != cudaSuccess) return -1;
        if (cudaMemset(p, 0, sizeof(g_wait_prof)) != cudaSuccess) return -1;
    }
    return 0;
}
#endif

size_t warp_kernel_smem_bytes(int head_dim) {
    return (head_dim == 128 ? SmemLayout<128>::kTotal : SmemLayout<64>::kTotal) + 1024;
}

cudaError_t configure_tc_kernel();

cudaError_t configure_attention_kernels() {
    cudaError_t e = configure_tc_kernel();
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(seg_attn_warp_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)warp_kernel_smem_bytes(128));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(seg_attn_warp_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)warp_kernel_smem_bytes(64));
}

cudaError_t launch_seg_attn_warp(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnArgs& a,
                                 cudaStream_t stream, bool after_tc) {
    if (a.grid_warp == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.grid_warp, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = warp_kernel_smem_bytes(a.head_dim);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = after_tc ? 1 : 0;
    if (a.head_dim == 128) return cudaLaunchKernelEx(&cfg, seg_attn_warp_kernel<128>, tm_k, tm_v, a);
    return cudaLaunchKernelEx(&cfg, seg_attn_warp_kernel<64>, tm_k, tm_v, a);
}

}  // namespace rksc
