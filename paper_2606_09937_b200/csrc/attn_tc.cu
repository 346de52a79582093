// Segment attention on the 5th-generation tensor cores (tcgen05 + TMEM) for work items with
// 17..128 stacked query rows and head_dim 128.
//
// All branches that share a segment, times the G query heads of a KV head, are stacked into the
// 128 rows of one MMA tile; a KV page staged in shared memory once then serves every sharing
// branch (the shared-prefix read that replaces the paper's per-branch copies of the prefix cache,
// Algorithm 1 line 3 / Section 2.2).  Here the product really is a dense contraction:
//   S[128 x 64]  = Q[128 x d] K^T        (tcgen05.mma, A = Q read from tensor memory, B = K slot, K-major,
//                                         in 128-byte-swizzled smem)
//   O[128 x d]  += P[128 x 64] V         (A = P read from tensor memory, B = V MN-major in smem)
// with Q, S, P and O in tensor memory.  One persistent CTA per SM, eleven warps:
//   warps 0-3 / 4-7  two softmax warpgroups; thread = one stacked row (TMEM lane).  They take
//                    alternate 64-token slots of an item, each with its own S and O accumulator and
//                    its own running (max, sum), merged at the end of the item.  Per slot: tcgen05.ld
//                    of the S row, scale + mask + online softmax in base 2, per-page softmax mass
//                    (log2, absolute) to global memory, P as bf16 back to tensor memory (tcgen05.st);
//                    O is rescaled in TMEM (tcgen05.ld / st) only when a running maximum of the warp moved.
//   warp 8           producer: claims work items from a global counter and streams their pages by
//                    TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast) into a five-slot
//                    ring, four pages per slot, with a header per slot that the other warps follow.
//   warps 9, 10      MMA issuers, one per warpgroup (one lane each; warp 9 also allocates TMEM): S of the
//                    warpgroup's next slot is issued before P V of its previous one, so S is waiting when
//                    the warpgroup comes out of its softmax and the tensor pipe runs under both softmaxes.
// Completion of MMAs is signalled with tcgen05.commit onto mbarriers (S ready, O ready / P free,
// ring slot free).  Every wait is bounded: on expiry the CTA records RKSC_ERR_DEVICE_TIMEOUT,
// stops issuing work, skips further waits, frees its TMEM and returns.
#include <cuda_bf16.h>

#include "kernels.h"

namespace rksc {

namespace {

constexpr int HD = 128;
constexpr int kSmWarps = 8;                       // softmax warps (two warpgroups)
constexpr int kProducerWarp = kSmWarps;           // 8
constexpr int kMmaWarp = kSmWarps + 1;            // 9 and 10: MMA issuers of warpgroup 0 and 1
constexpr int kTcThreads = (kSmWarps + 3) * 32;   // 352
constexpr int kNS = 6;                            // ring slots
constexpr int kSlotTokens = 64;                   // 4 pages
constexpr int kKBytes = kSlotTokens * HD * 2;     // K (or V) of a slot: [half][64 tokens][128 B] = 16 KiB
constexpr int kSlotBytes = 2 * kKBytes;
constexpr int kRingBytes = kNS * kSlotBytes;      // 192 KiB
constexpr int kMlOff = kRingBytes;                // (m, l) exchange [2][128] float2
constexpr int kBarOff = kMlOff + 2 * 128 * 8;
// mbarriers
constexpr int kBarFull = 0;                       // [kNS]  producer -> everyone: slot landed (+ header)
constexpr int kBarEmpty = kBarFull + kNS;         // [kNS]  slot reusable: P V committed + 10 header readers
constexpr int kBarSFull = kBarEmpty + kNS;        // [2]    S of the warpgroup's slot is in TMEM
constexpr int kBarSFree = kBarSFull + 2;          // [2]    the warpgroup has copied S to registers
constexpr int kBarPFull = kBarSFree + 2;          // [2]    P of the slot is in tensor memory
constexpr int kBarODone = kBarPFull + 2;          // [2]    P V of the slot has completed
constexpr int kBarQFull = kBarODone + 2;          // Q tile of the item is in tensor memory
constexpr int kBarEpiA = kBarQFull + 1;           // item epilogue: (m, l) published
constexpr int kBarEpiB = kBarEpiA + 1;            // item epilogue: accumulators read
constexpr int kNumBars = kBarEpiB + 1;
constexpr int kHdrOff = kBarOff + ((kNumBars * 8 + 15) / 16) * 16;
constexpr int kTmemPtrOff = kHdrOff + kNS * 64;
constexpr int kFlagOff = kTmemPtrOff + 16;
constexpr int kSmemTotal = kFlagOff + 16;
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;                     // S[wg]: 64 fp32 columns at 64*wg
constexpr uint32_t kColO = 128;                   // O[wg]: 128 fp32 columns at 128 + 128*wg
constexpr uint32_t kColP = 384;                   // P[wg]: 64 bf16 = 32 columns at 384 + 32*wg
constexpr uint32_t kColQ = 448;                   // Q: 128 bf16 per row = 64 columns (half wg written by warpgroup wg)
constexpr float kRescaleStep = 8.f;               // O is rescaled only when a row's max moved by more than 2^8

struct __align__(16) SlotHeader {
    int32_t item;        // index of the work item, -1: no more work
    int32_t group;       // position of this slot within the item (0 = first)
    int32_t num_pages;   // pages staged in this slot (1..4)
    int32_t last;        // 1 on the item's last slot
    WorkItem it;
    int32_t num_groups;  // slots of the item
    int32_t pad;
};
static_assert(sizeof(SlotHeader) == 64, "SlotHeader is 64 bytes");

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
// Bounded wait: gives up after 2^32 SM cycles (about two seconds).
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const long long t0 = clock64();
    for (;;) {
        if (mbar_try_wait(bar, parity)) return true;
        if (clock64() - t0 > (1ll << 32)) return false;
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar)
        : "memory");
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

// ---- tcgen05 ----
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// Shared-memory matrix descriptor: 128-byte swizzle, 8-row groups `sbo` bytes apart, 64-element
// blocks along the leading (MN) dimension `lbo` bytes apart (only used by the MN-major operand).
__device__ __forceinline__ uint64_t smem_desc(uint32_t saddr, uint32_t lbo, uint32_t sbo) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)((lbo >> 4) & 0x3FFFu) << 16;
    d |= (uint64_t)((sbo >> 4) & 0x3FFFu) << 32;
    d |= (uint64_t)1 << 46;   // descriptor version of this architecture
    d |= (uint64_t)2 << 61;   // SWIZZLE_128B
    return d;
}
// Instruction descriptor, kind::f16: fp32 accumulate, bf16 x bf16, M = 128.
__host__ __device__ constexpr uint32_t instr_desc(int n, int b_mn_major) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)b_mn_major << 16) | ((uint32_t)(n >> 3) << 17) |
           ((uint32_t)(128 >> 4) << 24);
}
// A operand (128 x 16 bf16, two values per 32-bit column) read from tensor memory
__device__ __forceinline__ void umma_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// 32 consecutive columns of this thread's TMEM lane
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
          "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
          "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
        : "r"(taddr)
        : "memory");
}
__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&r)[32]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16, "
        "%17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31, %32};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]),
          "r"(r[8]), "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15]),
          "r"(r[16]), "r"(r[17]), "r"(r[18]), "r"(r[19]), "r"(r[20]), "r"(r[21]), "r"(r[22]), "r"(r[23]),
          "r"(r[24]), "r"(r[25]), "r"(r[26]), "r"(r[27]), "r"(r[28]), "r"(r[29]), "r"(r[30]), "r"(r[31])
        : "memory");
}
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

#ifdef RKSC_WAIT_PROFILE
// Development aid: cycles per CTA spent in the waits of the MMA lane ([0..4]: total, slot landed,
// S buffer free, P ready, Q ready) and of softmax warp 0 ([8..15]: total, slot landed, S ready,
// previous P V done, epilogue A, epilogue B, slots, items).
__device__ unsigned long long g_tc_prof[384][16];
#define TCPROF_DECL unsigned long long tcp[8] = {0, 0, 0, 0, 0, 0, 0, 0}; const long long tcp_begin = clock64()
#define TCPROF_WAIT(i, stmt) { const long long _t = clock64(); stmt; tcp[i] += (unsigned long long)(clock64() - _t); }
#define TCPROF_MARK(i) { const long long _n = clock64(); tcq[i] += (unsigned long long)(_n - tcq_t); tcq_t = _n; }
#define TCPROF_FLUSH(base) { tcp[0] = (unsigned long long)(clock64() - tcp_begin); for (int _i = 0; _i < 8; ++_i) g_tc_prof[blockIdx.x][base + _i] = tcp[_i]; }
#else
#define TCPROF_DECL
#define TCPROF_WAIT(i, stmt) stmt
#define TCPROF_MARK(i)
#define TCPROF_FLUSH(base)
#endif

__global__ void __launch_bounds__(kTcThreads, 1)
seg_attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const AttnArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + kBarOff;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    SlotHeader* s_hdr = reinterpret_cast<SlotHeader*>(smem + kHdrOff);
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + kTmemPtrOff);
    volatile int32_t* s_abort = reinterpret_cast<volatile int32_t*>(smem + kFlagOff);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < kNS; ++i) {
            mbar_init(bar(kBarFull + i), 1);
            mbar_init(bar(kBarEmpty + i), 1 + kSmWarps + 2);   // P V commit, 8 softmax warps, 2 MMA issuers
        }
        for (int w = 0; w < 2; ++w) {
            mbar_init(bar(kBarSFull + w), 1);
            mbar_init(bar(kBarSFree + w), 4);
            mbar_init(bar(kBarPFull + w), 4);
            mbar_init(bar(kBarODone + w), 1);
        }
        mbar_init(bar(kBarQFull), kSmWarps);
        mbar_init(bar(kBarEpiA), kSmWarps);
        mbar_init(bar(kBarEpiB), kSmWarps);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        // the kernels that follow on the stream may be made resident early; they wait themselves
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    }
    if (warp == kMmaWarp) {   // one warp allocates (and later frees) the tensor memory
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(sbase + kTmemPtrOff),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
        tc_fence_before();
    }
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = *s_tmem;

    auto wait_or_abort = [&](uint32_t b, uint32_t parity) {
        if (*s_abort) return;
        if (!mbar_wait(b, parity)) {
            *s_abort = 1;
            if (a.status) atomicExch(a.status, RKSC_ERR_DEVICE_TIMEOUT);
        }
    };

    if (warp == kProducerWarp) {
        // ------------------------------------ producer ------------------------------------
        auto claim = [&]() {
            int v = 0;
            if (lane == 0) v = atomicAdd(a.counters + 2, 1);
            return __shfl_sync(0xffffffffu, v, 0);
        };
        auto fetch_item = [&](int i) {
            WorkItem w{};
            if (i < a.num_tc_items) w = a.plan.items[i];
            return w;
        };
        auto fetch_ids = [&](const WorkItem& w, int first) {
            return (first + lane < w.num_pages) ? __ldg(a.plan.seg_blocks + w.page_begin + first + lane) : 0;
        };
        // One item is claimed ahead of the one being streamed (its descriptor and first page ids are
        // fetched while this one streams); claiming further ahead would starve other CTAs, there
        // being only a few of these long items per CTA.
        int seq = 0;
        int idx = claim();
        WorkItem it = fetch_item(idx);
        int ids = fetch_ids(it, 0);
        while (idx < a.num_tc_items && !*s_abort) {
            const int nidx = claim();
            const WorkItem nit = fetch_item(nidx);
            const int ngroups = (it.num_pages + 3) / 4;
            int ids_ahead = 0;
            for (int g = 0; g < ngroups; ++g, ++seq) {
                const int slot = seq % kNS;
                const int npg = min(4, it.num_pages - g * 4);
                if ((g & 7) == 0) ids_ahead = fetch_ids(it, (g + 8) * 4);
                const int page = __shfl_sync(0xffffffffu, ids, (g & 7) * 4 + (lane & 3));
                if ((g & 7) == 7) ids = ids_ahead;
                if (seq >= kNS) wait_or_abort(bar(kBarEmpty + slot), (uint32_t)(seq / kNS - 1) & 1u);
                if (*s_abort) break;
                const uint32_t full = bar(kBarFull + slot);
                if (lane == 0) {
                    SlotHeader h;
                    h.item = idx;
                    h.group = g;
                    h.num_pages = npg;
                    h.last = (g == ngroups - 1);
                    h.it = it;
                    h.num_groups = ngroups;
                    h.pad = 0;
                    s_hdr[slot] = h;
                    mbar_arrive_expect_tx(full, npg * 2 * (kBlock * HD * 2));
                }
                __syncwarp();
                if (lane < npg) {
                    const int y = (page * a.Hkv + it.kv_head) * kBlock;
                    const uint32_t kdst = sbase + slot * kSlotBytes + lane * 2048;
#pragma unroll
                    for (int hh = 0; hh < 2; ++hh) {
                        tma_load_2d(kdst + hh * 8192, &tm_k, hh * 64, y, full);
                        tma_load_2d(kdst + kKBytes + hh * 8192, &tm_v, hh * 64, y, full);
                    }
                }
            }
            idx = nidx;
            it = nit;
            ids = fetch_ids(it, 0);
        }
        {   // end marker
            const int slot = seq % kNS;
            if (seq >= kNS) wait_or_abort(bar(kBarEmpty + slot), (uint32_t)(seq / kNS - 1) & 1u);
            if (lane == 0) {
                s_hdr[slot].item = -1;
                mbar_arrive(bar(kBarFull + slot));
            }
        }
        if (lane == 0) {   // the last CTA to stop claiming rewinds the counters for the next launch
            __threadfence();
            const int done = atomicAdd(a.counters + 3, 1);
            if (done == (int)gridDim.x - 1) {
                a.counters[2] = 0;
                a.counters[3] = 0;
                __threadfence();
            }
        }
    } else if (warp >= kMmaWarp) {
        // ------------------------- MMA issuers: warp 9 for warpgroup 0, warp 10 for warpgroup 1 -------------------------
        // Each walks every slot header (to see item boundaries) and issues the MMAs of its own
        // warpgroup's slots: S of the next own slot goes out before P V of the previous one, so S
        // is ready by the time the warpgroup finishes its softmax.
        if (lane == 0) {
            constexpr uint32_t kIdescQK = instr_desc(kSlotTokens, 0);
            constexpr uint32_t kIdescPV = instr_desc(HD, 1);
            const int wg = warp - kMmaWarp;
            int c = 0;                   // own slots issued (all items)
            bool first_pv = true;
            int item_k = -1;
            int pend_slot = -1, pend_npg = 0, pend_c = 0;
            TCPROF_DECL;
            auto flush_pv = [&]() {
                if (pend_slot < 0) return;
                TCPROF_WAIT(3, wait_or_abort(bar(kBarPFull + wg), (uint32_t)pend_c & 1u));
                if (!*s_abort) {
                    tc_fence_after();
                    const uint32_t vbase = sbase + pend_slot * kSlotBytes + kKBytes;
                    TCPROF_WAIT(6, for (int j = 0; j < pend_npg; ++j) {
                        const uint64_t bd = smem_desc(vbase + j * 2048, 8192, 1024);
                        umma_ts(tmem + kColO + wg * 128, tmem + kColP + wg * 32 + j * 8, bd, kIdescPV,
                                (first_pv && j == 0) ? 0u : 1u);
                    });
                    first_pv = false;
                    TCPROF_WAIT(7, tc_commit(bar(kBarODone + wg));
                    tc_commit(bar(kBarEmpty + pend_slot)));
                }
                pend_slot = -1;
            };
            for (int seq = 0; !*s_abort; ++seq) {
                const int slot = seq % kNS;
                TCPROF_WAIT(1, wait_or_abort(bar(kBarFull + slot), (uint32_t)(seq / kNS) & 1u));
                if (*s_abort) break;
                const int4 hdr = *reinterpret_cast<const int4*>(&s_hdr[slot]);   // item, group, pages, last
                if (hdr.x < 0) break;
                const int g = hdr.y, npg = hdr.z;
                const bool own = (g & 1) == wg;
                // a slot of the other warpgroup is only looked at: hand the header back
                if (!own) mbar_arrive(bar(kBarEmpty + slot));
                if (g == 0) {
                    flush_pv();
                    ++item_k;
                    TCPROF_WAIT(4, wait_or_abort(bar(kBarQFull), (uint32_t)item_k & 1u));
                    if (*s_abort) break;
                    first_pv = true;
                }
                if (!own) continue;
                if (c > 0) TCPROF_WAIT(2, wait_or_abort(bar(kBarSFree + wg), (uint32_t)(c - 1) & 1u));
                if (*s_abort) break;
                tc_fence_after();
                const uint32_t kbase = sbase + slot * kSlotBytes;
                TCPROF_WAIT(5, for (int ks = 0; ks < HD / 16; ++ks) {
                    const uint64_t bd = smem_desc(kbase + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024);
                    umma_ts(tmem + kColS + wg * 64, tmem + kColQ + ks * 8, bd, kIdescQK, ks > 0 ? 1u : 0u);
                });
                tc_commit(bar(kBarSFull + wg));
                mbar_arrive(bar(kBarEmpty + slot));   // this issuer's share of the slot's release (the P V commit is another)
                flush_pv();   // P V of the previous own slot, after S of this one
                pend_slot = slot;
                pend_npg = npg;
                pend_c = c;
                ++c;
            }
            flush_pv();
            if (wg == 0) { TCPROF_FLUSH(0); }
        }
        __syncwarp();
    } else {
        // ------------------------------------ softmax warps ------------------------------------
        const int wg = warp >> 2, quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        const float scale_log2 = a.scale_log2;
        const int G = a.G;
        float2* s_ml = reinterpret_cast<float2*>(smem + kMlOff);

        int cwg = 0;        // slots this warpgroup has processed (all items)
        int citem = 0;      // ... in the current item
        int item_k = -1;
        WorkItem it{};
        int rows = 0;
        bool valid = false, warp_has_rows = false;
        int64_t mb = 0;
        float m = -INFINITY, l = 0.f;
        TCPROF_DECL;
#ifdef RKSC_WAIT_PROFILE
        unsigned long long tcq[8] = {0, 0, 0, 0, 0, 0, 0, 0};
        long long tcq_t = 0;
#endif

        for (int seq = 0;; ++seq) {
            const int slot = seq % kNS;
            TCPROF_WAIT(1, wait_or_abort(bar(kBarFull + slot), (uint32_t)(seq / kNS) & 1u));
            if (*s_abort) break;
            const int4 hdr = *reinterpret_cast<const int4*>(&s_hdr[slot]);   // item, group, pages, last
            if (hdr.x < 0) break;
            const int g = hdr.y, npg = hdr.z;
            int ngroups = 0;
            if (g == 0) {
                it = s_hdr[slot].it;
            }
            ngroups = s_hdr[slot].num_groups;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarEmpty + slot));   // header read

            if (g == 0) {
                // ---- new item: row bookkeeping and the Q tile ----
                ++item_k;
                rows = it.num_sharers * G;
                valid = row < rows;
                warp_has_rows = quad * 32 < rows;
                m = -INFINITY;
                l = 0.f;
                citem = 0;
                const uint4* qsrc = nullptr;
                if (valid) {
                    const Sharer sh = a.plan.sharers[it.sharer_begin + row / G];
                    const int h = it.kv_head * G + row % G;
                    mb = sh.mass_base + (int64_t)h * sh.nblk + it.seg_page_begin;
                    qsrc = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(a.q) +
                                                          ((size_t)sh.branch * a.Hq + h) * HD + wg * 64);
                }
                // this warpgroup stages half `wg` (64 of the 128 dims) of every row into the Q columns of
                // tensor memory: thread = row = TMEM lane, two bf16 per 32-bit column (A operand of Q K^T)
                {
                    uint32_t qr[32];
#pragma unroll
                    for (int c = 0; c < 8; ++c) {
                        uint4 v = make_uint4(0u, 0u, 0u, 0u);
                        if (valid) v = __ldg(qsrc + c);
                        qr[4 * c] = v.x;
                        qr[4 * c + 1] = v.y;
                        qr[4 * c + 2] = v.z;
                        qr[4 * c + 3] = v.w;
                    }
                    tmem_st32(lane_addr + kColQ + wg * 32, qr);
                    tmem_wait_st();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarQFull));
            }

            if ((g & 1) == wg) {
                // ---- this warpgroup's slot: S row -> softmax -> P row ----
                TCPROF_WAIT(2, wait_or_abort(bar(kBarSFull + wg), (uint32_t)cwg & 1u));
                if (*s_abort) break;
                tc_fence_after();
#ifdef RKSC_WAIT_PROFILE
                tcq_t = clock64();
#endif
                uint32_t sr[2][32];
                tmem_ld32(lane_addr + kColS + wg * 64, sr[0]);
                tmem_ld32(lane_addr + kColS + wg * 64 + 32, sr[1]);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarSFree + wg));
                TCPROF_MARK(0);

                const int nvalid = it.num_tokens - g * kSlotTokens;   // tokens of this slot that exist
                float mx = -INFINITY;
#ifdef RKSC_TC_SKIP_SOFTMAX
                mx = __uint_as_float(sr[0][0]) * 0.f;
#else
                if (warp_has_rows) {
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains instead of one
                    if (nvalid >= kSlotTokens) {
#pragma unroll
                        for (int j = 0; j < 64; ++j) {
                            const float v = __uint_as_float(sr[j >> 5][j & 31]) * scale_log2;
                            sr[j >> 5][j & 31] = __float_as_uint(v);
                            mx4[j & 3] = fmaxf(mx4[j & 3], v);
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 64; ++j) {
                            float v = __uint_as_float(sr[j >> 5][j & 31]) * scale_log2;
                            v = (j < nvalid) ? v : -INFINITY;
                            sr[j >> 5][j & 31] = __float_as_uint(v);
                            mx4[j & 3] = fmaxf(mx4[j & 3], v);
                        }
                    }
                    mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                }
#endif
                TCPROF_MARK(1);

                // Running maximum with slack: m is raised (and O, l rescaled) only when a row's maximum
                // moved up by more than kRescaleStep, so p = 2^(s - m) stays below 2^kRescaleStep and the
                // TMEM round trip of O is rare.  The first slot of the item just adopts its maximum.
                if (citem == 0) {
                    if (valid) m = mx;
                } else {
                    // the previous P V of this warpgroup must be complete before P is overwritten or O touched
                    TCPROF_WAIT(3, wait_or_abort(bar(kBarODone + wg), (uint32_t)(cwg - 1) & 1u));
                    if (*s_abort) break;
                    tc_fence_after();
                    const bool grew = valid && (mx > m + kRescaleStep);
                    if (__any_sync(0xffffffffu, grew)) {
                        const float alpha = grew ? fast_exp2(m - mx) : 1.f;
                        l *= alpha;
#pragma unroll 1
                        for (int c = 0; c < HD / 32; ++c) {
                            uint32_t o[32];
                            tmem_ld32(lane_addr + kColO + wg * 128 + c * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                            tmem_st32(lane_addr + kColO + wg * 128 + c * 32, o);
                        }
                        tmem_wait_st();
                        if (grew) m = mx;
                    }
                }
                TCPROF_MARK(2);

                float ps[4] = {0.f, 0.f, 0.f, 0.f};
#ifndef RKSC_TC_SKIP_SOFTMAX
                if (warp_has_rows) {
                    const float mm = valid ? m : 0.f;   // rows past the item's end hold zeros: harmless, never read
#pragma unroll
                    for (int j = 0; j < 64; ++j) {
                        const float p = fast_exp2(__uint_as_float(sr[j >> 5][j & 31]) - mm);
                        sr[j >> 5][j & 31] = __float_as_uint(p);
                        ps[j >> 4] += p;
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 64; ++j) sr[j >> 5][j & 31] = 0u;
                }
#endif
                l += (ps[0] + ps[1]) + (ps[2] + ps[3]);
                if (valid && a.block_mass != nullptr) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (j < npg) a.block_mass[mb + g * 4 + j] = m + fast_log2(ps[j]);
                }
                TCPROF_MARK(3);
                // P row as bf16 pairs into this warpgroup's P columns of tensor memory (A operand of P V)
                {
                    uint32_t pk[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const __nv_bfloat162 b2 = __floats2bfloat162_rn(__uint_as_float(sr[(2 * j) >> 5][(2 * j) & 31]),
                                                                        __uint_as_float(sr[(2 * j + 1) >> 5][(2 * j + 1) & 31]));
                        pk[j] = *reinterpret_cast<const uint32_t*>(&b2);
                    }
                    tmem_st32(lane_addr + kColP + wg * 32, pk);
                    tmem_wait_st();
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPFull + wg));
                TCPROF_MARK(4);
                ++cwg;
                ++citem;
            }

            if (!hdr.w) continue;

            // ---- item epilogue: merge the two warpgroups' states, write the partial ----
            if (citem > 0) {
                wait_or_abort(bar(kBarODone + wg), (uint32_t)(cwg - 1) & 1u);
                if (*s_abort) break;
                tc_fence_after();
            }
            s_ml[wg * 128 + row] = make_float2(m, l);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarEpiA));
            TCPROF_WAIT(4, wait_or_abort(bar(kBarEpiA), (uint32_t)item_k & 1u));
            if (*s_abort) break;
            tc_fence_after();
            {
                const float2 oth = s_ml[(1 - wg) * 128 + row];
                const bool have_self = citem > 0;                       // warpgroup-uniform
                const bool have_oth = ngroups > (1 - wg);               // the other warpgroup had a slot
                const float M = fmaxf(have_self ? m : -INFINITY, have_oth ? oth.x : -INFINITY);
                const float w_self = have_self ? fast_exp2(m - M) : 0.f;
                const float w_oth = have_oth ? fast_exp2(oth.x - M) : 0.f;
                const float L = w_self * l + w_oth * oth.y;
                const float inv = 1.f / L;
                const float c_self = w_self * inv, c_oth = w_oth * inv;
                float* dst = a.part_o + ((size_t)it.part_row_base + row) * HD + wg * 64;
#pragma unroll 1
                for (int hh = 0; hh < 2; ++hh) {
                    float acc[32];
#pragma unroll
                    for (int j = 0; j < 32; ++j) acc[j] = 0.f;
                    if (have_self) {
                        uint32_t o[32];
                        tmem_ld32(lane_addr + kColO + wg * 128 + wg * 64 + hh * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) acc[j] = c_self * __uint_as_float(o[j]);
                    }
                    if (have_oth) {
                        uint32_t o[32];
                        tmem_ld32(lane_addr + kColO + (1 - wg) * 128 + wg * 64 + hh * 32, o);
                        tmem_wait_ld();
#pragma unroll
                        for (int j = 0; j < 32; ++j) acc[j] += c_oth * __uint_as_float(o[j]);
                    }
                    if (valid) {
#pragma unroll
                        for (int j = 0; j < 8; ++j)
                            *reinterpret_cast<float4*>(dst + hh * 32 + j * 4) =
                                make_float4(acc[4 * j], acc[4 * j + 1], acc[4 * j + 2], acc[4 * j + 3]);
                    }
                }
                if (valid && wg == 0) a.part_lse[(size_t)it.part_row_base + row] = M + fast_log2(L);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarEpiB));
            TCPROF_WAIT(5, wait_or_abort(bar(kBarEpiB), (uint32_t)item_k & 1u));
            if (*s_abort) break;
        }
#ifdef RKSC_WAIT_PROFILE
        if (warp == 0 && lane == 0) {
            tcp[6] = (unsigned long long)cwg; tcp[7] = (unsigned long long)(item_k + 1); TCPROF_FLUSH(8);
            for (int _i = 0; _i < 8; ++_i) g_tc_prof[blockIdx.x + 128][_i] = tcq[_i];
        }
#endif
    }

    // ---- common exit: free the tensor memory once nobody uses it ----
    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
    }
}

}  // namespace

#ifdef RKSC_WAIT_PROFILE
extern "C" __attribute__((visibility("default"))) int rksc_debug_tc_profile(unsigned long long* host_out) {
    return cudaMemcpyFromSymbol(host_out, g_tc_prof, sizeof(g_tc_prof)) == cudaSuccess ? 0 : -1;
}
#endif

size_t tc_kernel_smem_bytes() { return kSmemTotal + 1024; }

cudaError_t configure_tc_kernel() {
    return cudaFuncSetAttribute(seg_attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)tc_kernel_smem_bytes());
}

cudaError_t launch_seg_attn_tc(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnArgs& a,
                               cudaStream_t stream) {
    if (a.grid_tc == 0) return cudaSuccess;
    seg_attn_tc_kernel<<<a.grid_tc, kTcThreads, tc_kernel_smem_bytes(), stream>>>(tm_k, tm_v, a);
    return cudaGetLastError();
}

}  // namespace rksc
