// Segment attention on the 5th-generation tensor cores (tcgen05 + TMEM) for work items with
// 9..128 stacked query rows and head_dim 128.
//
// All branches that share a segment, times the G query heads of a KV head, are stacked into the
// 128 rows of one MMA tile; a KV page staged in shared memory once then serves every sharing
// branch (the shared-prefix read that replaces the paper's per-branch copies of the prefix cache,
// Algorithm 1 line 3 / Section 2.2).  Here the product really is a dense contraction:
//   S[128 x 64]  = Q[128 x d] K^T        (tcgen05.mma, A = Q and B = K slot, both K-major in
//                                         128-byte-swizzled shared memory)
//   O[128 x d]  += P[128 x 64] V         (A = P read from tensor memory, B = V MN-major in smem)
// with S, P and O in tensor memory.  One persistent CTA per SM, sixteen warps in four warpgroups:
//   warps 0-3 / 4-7  two softmax warpgroups; thread = one stacked row (TMEM lane).  They take
//                    alternate 64-token slots, each with two S buffers, its own O accumulator and
//                    its own running (max, sum), merged at the end of the item.  Per slot: tcgen05.ld
//                    of the S row, scale + mask + online softmax in base 2, per-page softmax mass
//                    (log2, absolute) to global memory, P written over the same S buffer in two bf16
//                    parts (tcgen05.st); O is rescaled in TMEM only when a running maximum of the
//                    warp moved by more than 2^8.  A warpgroup's only wait per slot is "S ready".
//   warp 8           K producer: takes work items (the first by CTA index, then from a global counter),
//                    publishes their descriptors in a small item ring and streams the K half of their
//                    pages by TMA (cp.async.bulk.tensor, 128-byte swizzle, no multicast) into a
//                    four-slot K ring, four pages per slot.
//   warp 12          V producer: follows the item ring and streams the V halves into a four-slot V ring.
//                    (One warp issues TMA copies at about 2.8 TB/s device-wide at most; and K, needed
//                    two slots before a slot's softmax, and V, needed after it, would pin a common slot
//                    four slot times.)
//   warps 9, 10      Q K^T issuers, one per warpgroup (one lane each; warp 9 also allocates TMEM): S of
//                    the warpgroup's slot c is issued once its K has landed and P V of slot c - 2 has
//                    left the buffer, so S is waiting when the warpgroup comes out of its softmax.
//   warps 13, 14     P V issuers, one per warpgroup.  (One thread issues a tcgen05.mma only every
//                    100-150 cycles: a single issuer per warpgroup was busy the whole slot.)
//   warp 11          Q loader: an item ahead, gathers the item's stacked query rows into one of two
//                    swizzled Q tiles (cp.async) and each row's block-mass base into shared memory.
//   warp 15          idle (it completes the fourth warpgroup, so that registers can be re-divided:
//                    192 per softmax thread, 64 per helper thread).
// Completion of MMAs is signalled with tcgen05.commit onto mbarriers (S ready, P V done / S buffer
// free, ring slots free, Q tile free).  Every wait is bounded: on expiry the CTA records
// RKSC_ERR_DEVICE_TIMEOUT, stops issuing work, skips further waits, frees its TMEM and returns.
#include <cuda_bf16.h>

#include "kernels.h"

namespace rksc {

namespace {

constexpr int HD = 128;
constexpr int kSmWarps = 8;                       // softmax warps (two warpgroups)
constexpr int kProducerWarp = kSmWarps;           // 8
constexpr int kMmaWarp = kSmWarps + 1;            // 9 and 10: Q K^T issuers of warpgroup 0 and 1
constexpr int kQWarp = kSmWarps + 3;              // 11: Q loader
constexpr int kVWarp = kSmWarps + 4;              // 12: V producer
constexpr int kPvWarp = kSmWarps + 5;             // 13 and 14: P V issuers of warpgroup 0 and 1
constexpr int kTcThreads = (kSmWarps + 8) * 32;   // 512: four warpgroups (warp 15 idles), so that registers can be re-divided
constexpr int kNK = 4;                            // K ring slots (even: a slot always serves the same warpgroup)
constexpr int kNV = 4;                            // V ring slots (even)
constexpr int kNI = 4;                            // item ring entries
constexpr int kSlotTokens = 64;                   // 4 pages
constexpr int kKBytes = kSlotTokens * HD * 2;     // K (or V) of a slot: [half][64 tokens][128 B] = 16 KiB
constexpr int kVOff = kNK * kKBytes;
constexpr int kRingBytes = (kNK + kNV) * kKBytes; // 128 KiB
static_assert(kNK % 2 == 0 && kNV % 2 == 0, "ring geometry");
constexpr int kQOff = kRingBytes;                 // Q tiles [2 (item parity)][half][128 rows][128 B], 128-byte swizzle: 2 x 32 KiB
constexpr int kQBytes = 128 * HD * 2;
constexpr int kRowOff = kQOff + 2 * kQBytes;      // block-mass base of every row [2][128] int64
constexpr int kMlOff = kRowOff + 2 * 128 * 8;     // (m, l) exchange [2 (item parity)][2 (warpgroup)][128] float2
constexpr int kBarOff = kMlOff + 2 * 2 * 128 * 8;
// mbarriers
constexpr int kBarFullK = 0;                      // [kNK]  producer -> issuer: K of the slot landed
constexpr int kBarEmptyK = kBarFullK + kNK;       // [kNK]  K slot reusable: its Q K^T has completed
constexpr int kBarFullV = kBarEmptyK + kNK;       // [kNV]  V of the slot landed
constexpr int kBarEmptyV = kBarFullV + kNV;       // [kNV]  V slot reusable: its P V has completed
constexpr int kBarItemFull = kBarEmptyV + kNV;    // [kNI]  item descriptor published
constexpr int kBarItemEmpty = kBarItemFull + kNI; // [kNI]  ... read by the 8 softmax warps, 2 issuers, Q loader
constexpr int kBarQFull = kBarItemEmpty + kNI;    // [2]    Q tile and row bases of the item are in shared memory
constexpr int kBarQEmpty = kBarQFull + 2;         // [2]    every Q K^T of the item has completed (both issuers) and
                                                  //        the softmax warps have read their row bases
constexpr int kBarSFull = kBarQEmpty + 2;         // [2][2] S of the warpgroup's slot is in its buffer
constexpr int kBarPFull = kBarSFull + 4;          // [2][2] P of the slot is in the buffer
constexpr int kBarODone = kBarPFull + 4;          // [2]    P V of the warpgroup's slot has completed
constexpr int kBarPVDone = kBarODone + 2;         // [2][2] ... per S buffer: the buffer may take the next S
constexpr int kBarEpiA = kBarPVDone + 4;          //        item epilogue: (m, l) published
constexpr int kBarEpiB = kBarEpiA + 1;            //        item epilogue: accumulators read
constexpr int kNumBars = kBarEpiB + 1;
constexpr int kItemOff = kBarOff + ((kNumBars * 8 + 15) / 16) * 16;
constexpr int kTmemPtrOff = kItemOff + kNI * 64;
constexpr int kFlagOff = kTmemPtrOff + 16;
constexpr int kSmemTotal = kFlagOff + 16;
static_assert(kSmemTotal + 1024 <= 227 * 1024, "shared memory of the tcgen05 kernel");
constexpr uint32_t kTmemCols = 512;
constexpr uint32_t kColS = 0;                     // S[wg][buf]: 64 fp32 columns at 64 * (2 * wg + buf); P over its first 32
constexpr uint32_t kColO = 256;                   // O[wg]: 128 fp32 columns at 256 + 128 * wg
constexpr float kRescaleStep = 8.f;               // O is rescaled only when a row's max moved by more than 2^8

struct __align__(16) ItemHeader {
    int32_t item;        // index of the work item, -1: no more work
    int32_t num_groups;  // 64-token slots of the item
    int32_t pad0, pad1;
    WorkItem it;
    int32_t pad2, pad3;
};
static_assert(sizeof(ItemHeader) == 64, "ItemHeader is 64 bytes");

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
// The same with a suspend-time hint (nanoseconds): the thread sleeps in hardware until the phase
// completes or the time is up, instead of spinning - a dozen helper warps polling in a tight loop
// take issue slots from the softmax warps of their scheduler.
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
// Bounded wait: gives up after 2^32 SM cycles (about two seconds).
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
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
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

// A and B operands from shared memory
__device__ __forceinline__ void umma_ss(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}

#ifdef RKSC_WAIT_PROFILE
// Development aid: cycles one lane of each role spent in its waits.
__device__ unsigned long long g_tc_prof[160][32];
__device__ int g_tc_dbg[32][4];
__device__ int g_tc_dbg_n, g_tc_dbg_n2;
#define TCP_DECL unsigned long long tcp[8] = {0, 0, 0, 0, 0, 0, 0, 0}; const long long tcp_begin = clock64()
#define TCP_WAIT(i, stmt) { const long long _t = clock64(); stmt; tcp[i] += (unsigned long long)(clock64() - _t); }
#define TCP_FLUSH(base) { tcp[0] = (unsigned long long)(clock64() - tcp_begin); for (int _i = 0; _i < 8; ++_i) g_tc_prof[blockIdx.x][base + _i] = tcp[_i]; }
#else
#define TCP_DECL
#define TCP_WAIT(i, stmt) stmt
#define TCP_FLUSH(base)
#endif

__global__ void __launch_bounds__(kTcThreads, 1)
seg_attn_tc_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                   const AttnArgs a) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t sbase = smem_u32(smem);
    const uint32_t bars = sbase + kBarOff;
    auto bar = [&](int i) { return bars + 8u * (uint32_t)i; };
    ItemHeader* s_item = reinterpret_cast<ItemHeader*>(smem + kItemOff);
    int64_t* s_rowbase = reinterpret_cast<int64_t*>(smem + kRowOff);
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(smem + kTmemPtrOff);
    volatile int32_t* s_abort = reinterpret_cast<volatile int32_t*>(smem + kFlagOff);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    // The CTA's first item is item blockIdx.x.  The two warps that need it first ask for it before
    // anything else, so that the round trip passes behind the set-up below (the plan's arrays are
    // written by no kernel: reading them does not have to wait for the kernel before this one).
    WorkItem it_first{};
    if ((warp == kProducerWarp || warp == kQWarp) && (int)blockIdx.x < a.num_tc_items) it_first = work_item_of(a.plan.items, blockIdx.x, a.Hkv, a.G);
    if (tid == 0) {
        for (int i = 0; i < kNK; ++i) {
            mbar_init(bar(kBarFullK + i), 1);
            mbar_init(bar(kBarEmptyK + i), 1);
        }
        for (int i = 0; i < kNV; ++i) {
            mbar_init(bar(kBarFullV + i), 1);
            mbar_init(bar(kBarEmptyV + i), 1);
        }
        for (int i = 0; i < kNI; ++i) {
            mbar_init(bar(kBarItemFull + i), 1);
            mbar_init(bar(kBarItemEmpty + i), kSmWarps + 6);   // 8 softmax warps, 4 issuers, Q loader, V producer
        }
        for (int i = 0; i < 2; ++i) {
            mbar_init(bar(kBarQFull + i), 1);
            mbar_init(bar(kBarQEmpty + i), 2 + kSmWarps);
        }
        for (int i = 0; i < 4; ++i) {
            mbar_init(bar(kBarSFull + i), 1);
            mbar_init(bar(kBarPFull + i), 4);
        }
        mbar_init(bar(kBarODone + 0), 1);
        mbar_init(bar(kBarODone + 1), 1);
        for (int i = 0; i < 4; ++i) mbar_init(bar(kBarPVDone + i), 1);
        mbar_init(bar(kBarEpiA), kSmWarps);
        mbar_init(bar(kBarEpiB), kSmWarps);
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
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
    // Launched with programmatic stream serialisation: everything above (barriers, tensor memory) may
    // run while the kernel before this one on the stream is still draining; nothing below, which reads
    // what that kernel may have written (queries, pool, claim counters) and writes what it may still
    // read (partial results, masses), starts before it has completed.  Only then may the kernels after
    // this one be made resident: the warp-MMA kernel does not wait at its start.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (tid == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    auto wait_or_abort = [&](uint32_t b, uint32_t parity) {
        if (*s_abort) return;
        if (!mbar_wait(b, parity)) {
#ifdef RKSC_WAIT_PROFILE
            if (!*s_abort && atomicAdd(&g_tc_dbg_n, 1) < 32) {
                const int k_ = atomicAdd(&g_tc_dbg_n2, 1);
                if (k_ < 32) { g_tc_dbg[k_][0] = (b - bars) / 8; g_tc_dbg[k_][1] = parity; g_tc_dbg[k_][2] = warp; g_tc_dbg[k_][3] = blockIdx.x; }
            }
#endif
            *s_abort = 1;
            if (a.status) atomicExch(a.status, RKSC_ERR_DEVICE_TIMEOUT);
        }
    };

    // 512 threads leave 128 registers each; the two softmax warpgroups need more and the two
    // warpgroups of helper warps much less
    if (warp >= kSmWarps) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 64;" ::: "memory");
    if (warp == kProducerWarp) {
        // ------------------------------------ producer ------------------------------------
        // CTA i starts with item i (no round trip to the counter before the first load); the counter
        // hands out the items after the first gridDim.x
        auto claim = [&]() {
            int v = 0;
            if (lane == 0) v = (int)gridDim.x + atomicAdd(a.counters + 2, 1);
            return __shfl_sync(0xffffffffu, v, 0);
        };
        auto fetch_item = [&](int i) {
            WorkItem w{};
            if (i < a.num_tc_items) w = work_item_of(a.plan.items, i, a.Hkv, a.G);
            return w;
        };
        auto fetch_ids = [&](const WorkItem& w, int first) {
            return (first + lane < w.num_pages) ? __ldg(a.plan.seg_blocks + w.page_begin + first + lane) : 0;
        };
        TCP_DECL;
        int nitem = 0;   // item descriptors published
        auto publish = [&](int idx, const WorkItem& w) {
            const int e = nitem % kNI;
            if (nitem >= kNI) wait_or_abort(bar(kBarItemEmpty + e), (uint32_t)(nitem / kNI - 1) & 1u);
            if (lane == 0) {
                ItemHeader h{};
                h.item = idx < a.num_tc_items ? idx : -1;
                h.num_groups = (w.num_pages + 3) / 4;
                h.it = w;
                s_item[e] = h;
                mbar_arrive(bar(kBarItemFull + e));
            }
            __syncwarp();
            ++nitem;
        };
        // One item is claimed ahead of the one being streamed (its descriptor is published, so the Q
        // loader can fetch its rows, and its first page ids are fetched while this one streams);
        // claiming further ahead would starve other CTAs, there being only a few of these long
        // items per CTA.
        // K and V travel in rings of their own, each fed by its own warp (one warp cannot issue TMA
        // copies fast enough for the whole stream): K of a slot is needed two slots before its softmax
        // starts and is free again as soon as Q K^T has run, V is needed after the softmax.
        const uint64_t kv_policy = l2_evict_first_policy();
        int seq = 0;
        int idx = (int)blockIdx.x;
        WorkItem it = it_first;
        publish(idx, it);
        int ids = fetch_ids(it, 0);
        while (idx < a.num_tc_items && !*s_abort) {
            const int nidx = claim();
            const WorkItem nit = fetch_item(nidx);
            publish(nidx, nit);     // past the last item this is the end marker
            const int ngroups = (it.num_pages + 3) / 4;
            int ids_ahead = 0;
            for (int g = 0; g < ngroups; ++g, ++seq) {
                const int kslot = seq % kNK;
                const int npg = min(4, it.num_pages - g * 4);
                if ((g & 7) == 0) ids_ahead = fetch_ids(it, (g + 8) * 4);
                // lane = 2 * page + half
                const int page = __shfl_sync(0xffffffffu, ids, (g & 7) * 4 + ((lane >> 1) & 3));
                if ((g & 7) == 7) ids = ids_ahead;
                if (seq >= kNK) TCP_WAIT(1, wait_or_abort(bar(kBarEmptyK + kslot), (uint32_t)(seq / kNK - 1) & 1u));
                if (*s_abort) break;
                const uint32_t full = bar(kBarFullK + kslot);
                if (lane == 0) mbar_arrive_expect_tx(full, npg * (kBlock * HD * 2));
                __syncwarp();
                if (lane < npg * 2) {
                    const int y = (page * a.Hkv + it.kv_head) * kBlock;
                    tma_load_2d(sbase + kslot * kKBytes + (lane >> 1) * 2048 + (lane & 1) * 8192, &tm_k, (lane & 1) * 64, y, full, kv_policy);
                }
            }
            idx = nidx;
            it = nit;
            ids = fetch_ids(it, 0);
        }
        if (lane == 0) { TCP_FLUSH(0); }
        if (lane == 0) {   // the last CTA to stop claiming rewinds the counters for the next launch
            __threadfence();
            const int done = atomicAdd(a.counters + 3, 1);
            if (done == (int)gridDim.x - 1) {
                a.counters[2] = 0;
                a.counters[3] = 0;
                __threadfence();
            }
        }
    } else if (warp == kVWarp) {
        // ------------------------------ V producer ------------------------------
        // Follows the item ring and streams the V half of every slot (one warp cannot issue TMA
        // copies fast enough for both halves).
        const int nring = kNV;
        const int bfull = kBarFullV, bempty = kBarEmptyV;
        const uint32_t ring = sbase + kVOff;
        const CUtensorMap* tm = &tm_v;
        const uint64_t kv_policy = l2_evict_first_policy();
        int seq = 0;
        for (int k = 0; !*s_abort; ++k) {
            const int e = k % kNI;
            wait_or_abort(bar(kBarItemFull + e), (uint32_t)(k / kNI) & 1u);
            if (*s_abort) break;
            const int item = s_item[e].item;
            const int page_begin = s_item[e].it.page_begin, num_pages = s_item[e].it.num_pages;
            const int kvh = s_item[e].it.kv_head;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarItemEmpty + e));
            if (item < 0) break;
            auto fetch_ids = [&](int first) {
                return (first + lane < num_pages) ? __ldg(a.plan.seg_blocks + page_begin + first + lane) : 0;
            };
            const int ngroups = (num_pages + 3) / 4;
            int ids = fetch_ids(0), ids_ahead = 0;
            for (int g = 0; g < ngroups; ++g, ++seq) {
                const int slot = seq % nring;
                const int npg = min(4, num_pages - g * 4);
                if ((g & 7) == 0) ids_ahead = fetch_ids((g + 8) * 4);
                const int page = __shfl_sync(0xffffffffu, ids, (g & 7) * 4 + ((lane >> 1) & 3));   // lane = 2 * page + half
                if ((g & 7) == 7) ids = ids_ahead;
                if (seq >= nring) wait_or_abort(bar(bempty + slot), (uint32_t)(seq / nring - 1) & 1u);
                if (*s_abort) break;
                const uint32_t full = bar(bfull + slot);
                if (lane == 0) mbar_arrive_expect_tx(full, npg * (kBlock * HD * 2));
                __syncwarp();
                if (lane < npg * 2) {
                    const int y = (page * a.Hkv + kvh) * kBlock;
                    tma_load_2d(ring + slot * kKBytes + (lane >> 1) * 2048 + (lane & 1) * 8192, tm, (lane & 1) * 64, y, full, kv_policy);
                }
            }
        }
    } else if (warp == kQWarp) {
        // ------------------------------------ Q loader ------------------------------------
        // Row r of the tile <-> (sharer r / G, head r % G of the item's KV head).  16-byte chunk c of a
        // row goes to half c / 8, at chunk (c % 8) ^ (r % 8) of the row's 128 bytes (the 128-byte
        // swizzle the MMA's shared-memory descriptor expects).
        const int G = a.G;
        // the CTA's first item is item blockIdx.x: fetched here, alongside the producer's own fetch,
        // so that its sharers and query rows are on their way before the producer has published it
        const WorkItem it0 = it_first;
        for (int k = 0; !*s_abort; ++k) {
            const int e = k % kNI;
            Sharer sh[4];
            if (k == 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = lane + 32 * i;
                    sh[i] = Sharer{};
                    if (r < it0.num_sharers * G) sh[i] = a.plan.sharers[it0.sharer_begin + r / G];
                }
            }
            wait_or_abort(bar(kBarItemFull + e), (uint32_t)(k / kNI) & 1u);
            if (*s_abort) break;
            const int item = s_item[e].item;
            const WorkItem it = s_item[e].it;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarItemEmpty + e));
            if (item < 0) break;
            const int rows = it.num_sharers * G;
            // the sharers of this lane's four rows, fetched before the wait below
            if (k > 0) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int r = lane + 32 * i;
                    sh[i] = Sharer{};
                    if (r < rows) sh[i] = a.plan.sharers[it.sharer_begin + r / G];
                }
            }
            // this Q tile is free once every Q K^T of the item before the previous one has completed
            // and the softmax warps have read that item's row bases
            if (k >= 2) wait_or_abort(bar(kBarQEmpty + (k & 1)), (uint32_t)((k >> 1) - 1) & 1u);
            if (*s_abort) break;
            const uint32_t qdst = sbase + kQOff + (k & 1) * kQBytes;
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int r = lane + 32 * i;
                const uint32_t rowdst = qdst + r * 128;
                if (r < rows) {
                    const int h = it.kv_head * G + r % G;
                    s_rowbase[(k & 1) * 128 + r] = sh[i].mass_base + (int64_t)h * sh[i].nblk + it.seg_page_begin;
                    const uint4* src = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(a.q) +
                                                                      ((size_t)sh[i].branch * a.Hq + h) * HD);
#pragma unroll
                    for (int c = 0; c < 16; ++c)
                        cp_async16(rowdst + (c >> 3) * 16384 + (((c & 7) ^ (r & 7)) << 4), src + c);
                } else {
                    s_rowbase[(k & 1) * 128 + r] = 0;
#pragma unroll
                    for (int c = 0; c < 16; ++c)
                        *reinterpret_cast<uint4*>(smem + kQOff + (k & 1) * kQBytes + r * 128 + (c >> 3) * 16384 + (c & 7) * 16) =
                            make_uint4(0u, 0u, 0u, 0u);
                }
            }
            asm volatile("cp.async.wait_all;" ::: "memory");
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> the MMA's reads
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQFull + (k & 1)));
        }
    } else if (warp == kMmaWarp || warp == kMmaWarp + 1) {
        // ------------------------- Q K^T issuers: warp 9 for warpgroup 0, warp 10 for warpgroup 1 -------------------------
        // Slot number seq (counted over all items of the CTA) belongs to warpgroup seq % 2 (the rings
        // have an even number of slots, so a ring slot always serves the same warpgroup).  One thread
        // issues MMAs too slowly to serve a warpgroup alone, so S and P V have an issuer each.  S of
        // own slot c goes into buffer c % 2 as soon as K has landed and P V of own slot c - 2, which
        // read P from that buffer, has completed: two slots ahead of the softmax.
        if (lane == 0) {
            constexpr uint32_t kIdescQK = instr_desc(kSlotTokens, 0);
            const int wg = warp - kMmaWarp;
            const uint32_t qbase0 = sbase + kQOff;
            int seq = 0;                 // slots seen (all items, both warpgroups)
            int c = 0;                   // own slots issued
            TCP_DECL;
            for (int k = 0; !*s_abort; ++k) {
                const int e = k % kNI;
                TCP_WAIT(3, wait_or_abort(bar(kBarItemFull + e), (uint32_t)(k / kNI) & 1u));
                if (*s_abort) break;
                const int item = s_item[e].item;
                const int ngroups = s_item[e].num_groups;
                mbar_arrive(bar(kBarItemEmpty + e));
                if (item < 0) break;
                TCP_WAIT(4, wait_or_abort(bar(kBarQFull + (k & 1)), (uint32_t)(k >> 1) & 1u));
                if (*s_abort) break;
                const uint32_t qbase = qbase0 + (k & 1) * kQBytes;
                for (int g = 0; g < ngroups; ++g, ++seq) {
                    if ((seq & 1) != wg) continue;
                    const int slot = seq % kNK;
                    if (c >= 2) TCP_WAIT(1, wait_or_abort(bar(kBarPVDone + wg * 2 + (c & 1)), (uint32_t)((c >> 1) - 1) & 1u));
                    TCP_WAIT(5, wait_or_abort(bar(kBarFullK + slot), (uint32_t)(seq / kNK) & 1u));
                    if (*s_abort) break;
                    tc_fence_after();
                    const uint32_t kbase = sbase + slot * kKBytes;
                    const uint32_t scol = tmem + kColS + (uint32_t)(wg * 2 + (c & 1)) * 64;
                    TCP_WAIT(6, for (int ks = 0; ks < HD / 16; ++ks) {
                        const uint64_t ad = smem_desc(qbase + (ks >> 2) * 16384 + (ks & 3) * 32, 16, 1024);
                        const uint64_t bd = smem_desc(kbase + (ks >> 2) * 8192 + (ks & 3) * 32, 16, 1024);
                        umma_ss(scol, ad, bd, kIdescQK, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(bar(kBarSFull + wg * 2 + (c & 1)));
                    tc_commit(bar(kBarEmptyK + slot)));   // K of the slot is free as soon as S is there
                    ++c;
                }
                if (*s_abort) break;
                tc_commit(bar(kBarQEmpty + (k & 1)));   // this issuer's Q K^T of the item (if any) have completed
            }
            TCP_FLUSH(8 + 8 * wg);
        }
        __syncwarp();
    } else if (warp == kPvWarp || warp == kPvWarp + 1) {
        // ------------------------- P V issuers: warp 13 for warpgroup 0, warp 14 for warpgroup 1 -------------------------
        if (lane == 0) {
            constexpr uint32_t kIdescPV = instr_desc(HD, 1);
            const int wg = warp - kPvWarp;
            int seq = 0, c = 0;
            for (int k = 0; !*s_abort; ++k) {
                const int e = k % kNI;
                wait_or_abort(bar(kBarItemFull + e), (uint32_t)(k / kNI) & 1u);
                if (*s_abort) break;
                const int item = s_item[e].item;
                const int ngroups = s_item[e].num_groups;
                const int num_pages = s_item[e].it.num_pages;
                mbar_arrive(bar(kBarItemEmpty + e));
                if (item < 0) break;
                bool first_own = true;
                for (int g = 0; g < ngroups; ++g, ++seq) {
                    if ((seq & 1) != wg) continue;
                    const int slot = seq % kNV;
                    const int npg = min(4, num_pages - g * 4);
                    wait_or_abort(bar(kBarPFull + wg * 2 + (c & 1)), (uint32_t)(c >> 1) & 1u);
                    // the first P V of an item overwrites O: both warpgroups must have read out the previous item
                    if (first_own && k > 0) wait_or_abort(bar(kBarEpiB), (uint32_t)(k - 1) & 1u);
                    wait_or_abort(bar(kBarFullV + slot), (uint32_t)(seq / kNV) & 1u);
                    if (*s_abort) break;
                    tc_fence_after();
                    const uint32_t vbase = sbase + kVOff + slot * kKBytes;
                    const uint32_t pcol = tmem + kColS + (uint32_t)(wg * 2 + (c & 1)) * 64;
                    for (int j = 0; j < npg; ++j) {
                        const uint64_t bd = smem_desc(vbase + j * 2048, 8192, 1024);
                        umma_ts(tmem + kColO + wg * 128, pcol + j * 8, bd, kIdescPV, (first_own && j == 0) ? 0u : 1u);
                        umma_ts(tmem + kColO + wg * 128, pcol + 32 + j * 8, bd, kIdescPV, 1u);   // the lower part of P
                    }
                    tc_commit(bar(kBarPVDone + wg * 2 + (c & 1)));
                    tc_commit(bar(kBarODone + wg));
                    tc_commit(bar(kBarEmptyV + slot));
                    first_own = false;
                    ++c;
                }
            }
        }
        __syncwarp();
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 192;" ::: "memory");
        // ------------------------------------ softmax warps ------------------------------------
        const int wg = warp >> 2, quad = warp & 3;
        const int row = quad * 32 + lane;
        const uint32_t lane_addr = tmem + ((uint32_t)(quad * 32) << 16);
        const float scale_log2 = a.scale_log2;
        const int G = a.G;
        float2* s_ml = reinterpret_cast<float2*>(smem + kMlOff);

        int seq = 0;        // slots seen (all items, both warpgroups)
        int c = 0;          // own slots processed (all items)
        TCP_DECL;

        for (int k = 0; !*s_abort; ++k) {
            const int e = k % kNI;
            TCP_WAIT(1, wait_or_abort(bar(kBarItemFull + e), (uint32_t)(k / kNI) & 1u));
            if (*s_abort) break;
            const int item = s_item[e].item;
            const int ngroups = s_item[e].num_groups;
            const int it_num_tokens = s_item[e].it.num_tokens, it_num_pages = s_item[e].it.num_pages;
            const int it_part_row_base = s_item[e].it.part_row_base;
            const int rows = s_item[e].it.num_sharers * G;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarItemEmpty + e));
            if (item < 0) break;
            // row bases of the item (written by the Q loader before it signals the Q tile)
            TCP_WAIT(2, wait_or_abort(bar(kBarQFull + (k & 1)), (uint32_t)(k >> 1) & 1u));
            if (*s_abort) break;
            const bool valid = row < rows;
            const bool warp_has_rows = quad * 32 < rows;
            const int64_t mb = s_rowbase[(k & 1) * 128 + row];
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarQEmpty + (k & 1)));   // row bases read
            float m = -INFINITY, l = 0.f;
            int citem = 0;      // own slots of this item

            for (int g = 0; g < ngroups; ++g, ++seq) {
                if ((seq & 1) != wg) continue;
                // ---- this warpgroup's slot: S row -> softmax -> P row ----
                const uint32_t scol = lane_addr + kColS + (uint32_t)(wg * 2 + (c & 1)) * 64;
                TCP_WAIT(3, wait_or_abort(bar(kBarSFull + wg * 2 + (c & 1)), (uint32_t)(c >> 1) & 1u));
                if (*s_abort) break;
                tc_fence_after();
                uint32_t sr[2][32];
                tmem_ld32(scol, sr[0]);
                tmem_ld32(scol + 32, sr[1]);
                tmem_wait_ld();

                const int nvalid = it_num_tokens - g * kSlotTokens;   // tokens of this slot that exist
                const int npg = min(4, it_num_pages - g * 4);
                float mx = -INFINITY;
                if (warp_has_rows) {
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};   // four chains instead of one
                    // the maximum is taken over the raw scores (the scale is positive) and scaled once; the
                    // scale itself is applied inside the exponent's multiply-add below
                    if (nvalid >= kSlotTokens) {
#pragma unroll
                        for (int j = 0; j < 64; ++j) mx4[j & 3] = fmaxf(mx4[j & 3], __uint_as_float(sr[j >> 5][j & 31]));
                    } else {
#pragma unroll
                        for (int j = 0; j < 64; ++j) {
                            const float v = (j < nvalid) ? __uint_as_float(sr[j >> 5][j & 31]) : -INFINITY;
                            sr[j >> 5][j & 31] = __float_as_uint(v);
                            mx4[j & 3] = fmaxf(mx4[j & 3], v);
                        }
                    }
                    mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * scale_log2;
                }

                // Running maximum with slack: m is raised (and O, l rescaled) only when a row's maximum
                // moved up by more than kRescaleStep, so p = 2^(s - m) stays below 2^kRescaleStep and the
                // TMEM round trip of O is rare.  The first slot of the item just adopts its maximum.
                if (citem == 0) {
                    if (valid) m = mx;
                } else {
                    const bool grew = valid && (mx > m + kRescaleStep);
                    if (__any_sync(0xffffffffu, grew)) {
                        // O must be at rest: P V of this warpgroup's previous slot has to be complete
                        wait_or_abort(bar(kBarODone + wg), (uint32_t)(c - 1) & 1u);
                        if (*s_abort) break;
                        tc_fence_after();
                        const float alpha = grew ? fast_exp2(m - mx) : 1.f;
                        l *= alpha;
#pragma unroll 1
                        for (int cc = 0; cc < HD / 32; ++cc) {
                            uint32_t o[32];
                            tmem_ld32(lane_addr + kColO + wg * 128 + cc * 32, o);
                            tmem_wait_ld();
#pragma unroll
                            for (int j = 0; j < 32; ++j) o[j] = __float_as_uint(__uint_as_float(o[j]) * alpha);
                            tmem_st32(lane_addr + kColO + wg * 128 + cc * 32, o);
                        }
                        tmem_wait_st();
                        if (grew) m = mx;
                    }
                }

                // p = 2^(s - m), its per-page sums, and the P row as bf16 pairs (A operand of P V) in two
                // parts: the upper 16 bits of p, and the upper 16 bits of the rest.  One bf16 alone carries
                // 2^-9 relative error into the output, more than its tolerance when few tokens hold most of
                // a row's mass; P V is accumulated over both parts.
                float ps[4] = {0.f, 0.f, 0.f, 0.f};
                uint32_t pk[32], pl[32];
                if (warp_has_rows) {
                    const float mm = valid ? m : 0.f;   // rows past the item's end: harmless, never read
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        const float p0 = fast_exp2(fmaf(__uint_as_float(sr[(2 * j) >> 5][(2 * j) & 31]), scale_log2, -mm));
                        const float p1 = fast_exp2(fmaf(__uint_as_float(sr[(2 * j + 1) >> 5][(2 * j + 1) & 31]), scale_log2, -mm));
                        ps[j >> 3] += p0;
                        ps[j >> 3] += p1;
                        const uint32_t h0 = __float_as_uint(p0) & 0xffff0000u, h1 = __float_as_uint(p1) & 0xffff0000u;
                        pk[j] = __byte_perm(h0, h1, 0x7632);   // (h1 upper half, h0 upper half)
                        // the rest, p - upper part (exact in fp32), cut to its own upper 16 bits: 2^-16 of p is lost
                        pl[j] = __byte_perm(__float_as_uint(p0 - __uint_as_float(h0)), __float_as_uint(p1 - __uint_as_float(h1)), 0x7632);
                    }
                } else {
#pragma unroll
                    for (int j = 0; j < 32; ++j) pk[j] = pl[j] = 0u;
                }
                // over the S buffer, whose 64 values are all in registers by now: upper parts in its
                // first 32 columns, lower parts in the other 32
                tmem_st32(scol, pk);
                tmem_st32(scol + 32, pl);
                l += (ps[0] + ps[1]) + (ps[2] + ps[3]);
                if (valid && a.block_mass != nullptr) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (j < npg) a.block_mass[mb + g * 4 + j] = m + fast_log2(ps[j]);
                }
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(kBarPFull + wg * 2 + (c & 1)));
                ++c;
                ++citem;
            }
            if (*s_abort) break;

            // ---- item epilogue: merge the two warpgroups' states, write the partial ----
            const bool have_self = citem > 0;                 // warpgroup-uniform
            const bool have_oth = ngroups - citem > 0;        // the other warpgroup had a slot
            if (have_self) {
                // O is read out once the P V of this warpgroup's last two slots have completed.  A wait on a
                // barrier's parity tells the current phase only from the one before it, and nothing orders the
                // softmax of the last slot after the P V of the slot before it (the barrier that counts every
                // P V could still be two phases back and let a wait for "the last one" through at once).  The
                // per-buffer barriers cannot be that far back: the scores of slot c - 1 (c - 2) were only
                // computed after P V of slot c - 3 (c - 4) had left their buffer.
                if (c >= 2) TCP_WAIT(4, wait_or_abort(bar(kBarPVDone + wg * 2 + ((c - 2) & 1)), (uint32_t)((c - 2) >> 1) & 1u));
                if (*s_abort) break;
                TCP_WAIT(4, wait_or_abort(bar(kBarPVDone + wg * 2 + ((c - 1) & 1)), (uint32_t)((c - 1) >> 1) & 1u));
                if (*s_abort) break;
                tc_fence_after();
            }
            s_ml[((k & 1) * 2 + wg) * 128 + row] = make_float2(m, l);
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarEpiA));
            TCP_WAIT(5, wait_or_abort(bar(kBarEpiA), (uint32_t)k & 1u));
            if (*s_abort) break;
            tc_fence_after();
            {
                // The two warpgroups hold the item's even and odd slots; which of them holds which depends on
                // how many slots this CTA ran before the item (items are claimed dynamically).  The two states
                // are therefore combined symmetrically - products rounded on their own, then one addition, no
                // fused multiply-add across the two - so that an item's partial result has the same bits
                // whichever CTA ran it after whatever.
                const float2 oth = s_ml[((k & 1) * 2 + (1 - wg)) * 128 + row];
                const float M = fmaxf(have_self ? m : -INFINITY, have_oth ? oth.x : -INFINITY);
                const float w_self = have_self ? fast_exp2(m - M) : 0.f;
                const float w_oth = have_oth ? fast_exp2(oth.x - M) : 0.f;
                const float L = __fadd_rn(__fmul_rn(w_self, l), __fmul_rn(w_oth, oth.y));
                const float inv = 1.f / L;
                const float c_self = w_self * inv, c_oth = w_oth * inv;
                float* dst = a.part_o + ((size_t)it_part_row_base + row) * HD + wg * 64;
#pragma unroll 1
                for (int q4 = 0; q4 < 4; ++q4) {
                    uint32_t os[16], oo[16];
                    if (have_self) tmem_ld16(lane_addr + kColO + wg * 128 + wg * 64 + q4 * 16, os);
                    if (have_oth) tmem_ld16(lane_addr + kColO + (1 - wg) * 128 + wg * 64 + q4 * 16, oo);
                    tmem_wait_ld();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        // both products rounded, then one addition: the same bits in either role
                        const float ps_ = have_self ? __fmul_rn(c_self, __uint_as_float(os[j])) : 0.f;
                        const float po_ = have_oth ? __fmul_rn(c_oth, __uint_as_float(oo[j])) : 0.f;
                        os[j] = __float_as_uint(__fadd_rn(ps_, po_));
                    }
                    if (valid) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            *reinterpret_cast<uint4*>(dst + q4 * 16 + j * 4) =
                                make_uint4(os[4 * j], os[4 * j + 1], os[4 * j + 2], os[4 * j + 3]);
                    }
                }
                if (valid && wg == 0) a.part_lse[(size_t)it_part_row_base + row] = M + fast_log2(L);
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(kBarEpiB));   // the issuers wait for this before the next item's first P V
        }
#ifdef RKSC_WAIT_PROFILE
        if (wg == 0 && quad == 0 && lane == 0) { tcp[6] = (unsigned long long)c; TCP_FLUSH(24); }
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
extern "C" __attribute__((visibility("default"))) int rksc_debug_tc_dbg(int* host_out) {
    return cudaMemcpyFromSymbol(host_out, g_tc_dbg, sizeof(g_tc_dbg)) == cudaSuccess ? 0 : -1;
}
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
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.grid_tc, 1, 1);
    cfg.blockDim = dim3(kTcThreads, 1, 1);
    cfg.dynamicSmemBytes = tc_kernel_smem_bytes();
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, seg_attn_tc_kernel, tm_k, tm_v, a);
}

}  // namespace rksc
