// Segment attention with warp-level MMA (stacked rows <= 64): persistent, warp-specialised.
//
// A work item is a chunk of one segment's KV pages for one KV head plus a block of the branches
// that share the segment.  The query rows of all those branches x the G query heads of the KV
// head are stacked into 16-row tiles, so a page staged in shared memory once serves every
// sharing branch (this is what replaces the paper's B physical copies of the prefix cache,
// Algorithm 1 line 3 / Section 2.2).
//
//   * Persistent CTAs (two per SM), each with a host-packed list of work items.
//   * Warp 4 is the producer: it walks the CTA's items and streams their pages, four pages
//     (K and V, 16 tokens each) per ring slot, by TMA (cp.async.bulk.tensor, 128-byte swizzle,
//     16 x 64 boxes) with one mbarrier per slot for arrival and one for release.  It runs ahead
//     across item boundaries, so the ring never drains between items.  No cluster multicast.
//   * Warps 0-3 are consumers.  With R stacked rows there are nrt = ceil(R/16) row tiles; the
//     warps are arranged as (row tile) x (page lane): PL = 4, 2 or 1 page lanes split the pages of
//     every slot among them, and the row-tile warps of a lane read the same staged page.
//   * Per page and warp: S = Q K^T by mma.sync m16n8k16 (bf16 in, fp32 out), online softmax in
//     base 2, P split into a bf16 high and low part (two MMAs) so that P V carries fp32-level
//     error, and the page's softmax mass written as log2 (absolute, independent of the running
//     maximum) for the merge kernel to normalise.
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
__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait: gives up after about two seconds.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_timer_ns() - t0 > 2000000000ull) return false;
    }
}
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void consumer_bar_sync() {   // named barrier of the four consumer warps
    asm volatile("bar.sync 1, %0;" ::"n"(kCW * 32) : "memory");
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
    static constexpr int kFlagOff = kBarOff + 2 * kNS * 8;
    static constexpr int kTotal = kFlagOff + 16;
};

template <int HD>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
seg_attn_warp_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                     const AttnArgs a) {
    using SL = SmemLayout<HD>;
    constexpr int KS = HD / 16;      // k-steps of Q K^T
    constexpr int NT = HD / 8;       // n-tiles of P V
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const uint32_t ring = smem_u32(smem);
    const uint32_t bar_full = ring + SL::kBarOff;
    const uint32_t bar_empty = bar_full + kNS * 8;
    volatile int32_t* s_abort = reinterpret_cast<volatile int32_t*>(smem + SL::kFlagOff);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    if (tid == 0) {
        for (int i = 0; i < kNS; ++i) {
            mbar_init(bar_full + 8 * i, 1);
            mbar_init(bar_empty + 8 * i, kCW);
        }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    const int item_lo = a.plan.cta_item_off[blockIdx.x], item_hi = a.plan.cta_item_off[blockIdx.x + 1];

    auto wait_or_abort = [&](uint32_t bar, uint32_t parity) {
        if (*s_abort) return;
        if (!mbar_wait(bar, parity)) {
            *s_abort = 1;
            if (a.status) atomicExch(a.status, RKSC_ERR_DEVICE_TIMEOUT);
        }
    };

    if (warp == kCW) {
        // ------------------------------ producer warp ------------------------------
        int seq = 0;
        for (int k = item_lo; k < item_hi; ++k) {
            const WorkItem it = a.plan.items[a.plan.cta_items[k]];
            const int ngroups = (it.num_pages + kSP - 1) / kSP;
            for (int g = 0; g < ngroups; ++g, ++seq) {
                const int slot = seq % kNS;
                const int npg = min(kSP, it.num_pages - g * kSP);
                int page = 0;
                if (lane < npg) page = __ldg(a.plan.seg_blocks + it.page_begin + g * kSP + lane);
                if (seq >= kNS) wait_or_abort(bar_empty + 8 * slot, (uint32_t)(seq / kNS - 1) & 1u);
                if (*s_abort) break;
                const uint32_t bar = bar_full + 8 * slot;
                if (lane == 0) mbar_arrive_expect_tx(bar, npg * SL::kPage);
                __syncwarp();
                if (lane < npg) {
                    const int y = (page * a.Hkv + it.kv_head) * kBlock;
                    const uint32_t dst = ring + slot * SL::kSlot + lane * SL::kPage;
#pragma unroll
                    for (int hh = 0; hh < HD / 64; ++hh) {
                        tma_load_2d(dst + hh * 2048, &tm_k, hh * 64, y, bar);
                        tma_load_2d(dst + SL::kTile + hh * 2048, &tm_v, hh * 64, y, bar);
                    }
                }
            }
            if (*s_abort) break;
        }
        return;
    }

    // -------------------------------- consumer warps --------------------------------
    const int g4 = lane >> 2, t = lane & 3;
    // per-lane constants of the ldmatrix addresses
    const int k_tok = ((lane >> 4) << 3) + (lane & 7);       // K: token row this lane points at
    const int k_chunk = (lane >> 3) & 1;                     //    +1 chunk for the upper 8 of k
    const int v_tok = (((lane >> 3) & 1) << 3) + (lane & 7); // V: token row
    const int v_chunk = lane >> 4;                           //    +1 chunk for the next n-tile
    const uint32_t k_lane_off = k_tok * 128;
    const uint32_t v_lane_off = v_tok * 128;
    const float scale_log2 = a.scale_log2;
    const int G = a.G;
    float* scr = reinterpret_cast<float*>(smem + SL::kScrOff);
    float* s_m = reinterpret_cast<float*>(smem + SL::kMlOff);
    float* s_l = s_m + kCW * 16;

    int seq = 0;
    for (int k = item_lo; k < item_hi; ++k) {
        const WorkItem it = a.plan.items[a.plan.cta_items[k]];
        const int kvh = it.kv_head;
        const int rows = it.num_sharers * G;
        const int nrt = (rows + 15) >> 4;               // row tiles in use: 1..4
        const int nrtp = (nrt == 3) ? 4 : nrt;          // warps per page lane: 1, 2 or 4
        const int PL = kCW / nrtp;                      // page lanes
        const int rt = warp % nrtp, pl = warp / nrtp;
        const bool active = rt < nrt;

        // rows of this thread: r0 = rt*16 + g4 and r0 + 8
        const int r0 = rt * 16 + g4, r1 = r0 + 8;
        const bool v0 = active && r0 < rows, v1 = active && r1 < rows;
        int64_t mb0 = 0, mb1 = 0;
        uint32_t qf[KS][4];
        {
            const uint32_t* q0 = nullptr;
            const uint32_t* q1 = nullptr;
            if (v0) {
                const Sharer sh = a.plan.sharers[it.sharer_begin + r0 / G];
                const int h = kvh * G + r0 % G;
                q0 = reinterpret_cast<const uint32_t*>(a.q) + ((size_t)sh.branch * a.Hq + h) * (HD / 2);
                mb0 = sh.mass_base + (int64_t)h * sh.nblk + it.seg_page_begin;
            }
            if (v1) {
                const Sharer sh = a.plan.sharers[it.sharer_begin + r1 / G];
                const int h = kvh * G + r1 % G;
                q1 = reinterpret_cast<const uint32_t*>(a.q) + ((size_t)sh.branch * a.Hq + h) * (HD / 2);
                mb1 = sh.mass_base + (int64_t)h * sh.nblk + it.seg_page_begin;
            }
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qf[ks][0] = v0 ? __ldg(q0 + ks * 8 + t) : 0u;
                qf[ks][2] = v0 ? __ldg(q0 + ks * 8 + 4 + t) : 0u;
                qf[ks][1] = v1 ? __ldg(q1 + ks * 8 + t) : 0u;
                qf[ks][3] = v1 ? __ldg(q1 + ks * 8 + 4 + t) : 0u;
            }
        }

        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[NT][4];
#pragma unroll
        for (int n = 0; n < NT; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

        const int ngroups = (it.num_pages + kSP - 1) / kSP;
        for (int g = 0; g < ngroups; ++g, ++seq) {
            const int slot = seq % kNS;
            wait_or_abort(bar_full + 8 * slot, (uint32_t)(seq / kNS) & 1u);
            const int npg = min(kSP, it.num_pages - g * kSP);
            if (active) {
                for (int j = pl; j < npg; j += PL) {
                    const uint32_t kb = ring + slot * SL::kSlot + j * SL::kPage;
                    const uint32_t vb = kb + SL::kTile;
                    const int pi = g * kSP + j;                   // page index within the item
                    const int nv = it.num_tokens - pi * kBlock;   // valid tokens: >= 1, >= 16 if full

                    // S = Q K^T for 16 rows x 16 tokens
                    float s[2][4] = {{0.f, 0.f, 0.f, 0.f}, {0.f, 0.f, 0.f, 0.f}};
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        const int chunk = ((ks * 2) & 7) + k_chunk;
                        const uint32_t addr = kb + (ks >> 2) * 2048 + k_lane_off + ((chunk ^ (k_tok & 7)) << 4);
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
#pragma unroll
                    for (int n = 0; n < NT; ++n) {
                        o[n][0] *= al0;
                        o[n][1] *= al0;
                        o[n][2] *= al1;
                        o[n][3] *= al1;
                    }
                    // O += P V, P as bf16 high + low parts
                    uint32_t phi[4], plo[4];
                    split_pack(p[0][0], p[0][1], phi[0], plo[0]);
                    split_pack(p[0][2], p[0][3], phi[1], plo[1]);
                    split_pack(p[1][0], p[1][1], phi[2], plo[2]);
                    split_pack(p[1][2], p[1][3], phi[3], plo[3]);
#pragma unroll
                    for (int np = 0; np < NT / 2; ++np) {
                        const int chunk = ((np * 2) & 7) + v_chunk;
                        const uint32_t addr = vb + (np >> 2) * 2048 + v_lane_off + ((chunk ^ (v_tok & 7)) << 4);
                        uint32_t bv[4];
                        ldmatrix_x4_trans(addr, bv);
                        mma_bf16(o[2 * np], phi, bv[0], bv[1]);
                        mma_bf16(o[2 * np], plo, bv[0], bv[1]);
                        mma_bf16(o[2 * np + 1], phi, bv[2], bv[3]);
                        mma_bf16(o[2 * np + 1], plo, bv[2], bv[3]);
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_empty + 8 * slot);
        }

        // ---- item epilogue: merge the page lanes, write the partial (normalised O, log2-sum-exp) ----
        const size_t prow0 = (size_t)it.part_row_base;
        if (PL == 1) {
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
            // PL = 2 or 4 page lanes hold partial states of the same rows (all four warps are active)
            if (t == 0) {
                s_m[warp * 16 + g4] = m0;
                s_l[warp * 16 + g4] = l0;
                s_m[warp * 16 + g4 + 8] = m1;
                s_l[warp * 16 + g4 + 8] = l1;
            }
            float* my = scr + warp * (16 * SL::kScrRow);
            const int ctid = tid;   // 0..127 among the consumers
#pragma unroll
            for (int c = 0; c < HD / 32; ++c) {
#pragma unroll
                for (int n = 0; n < 4; ++n) {
                    *reinterpret_cast<float2*>(my + g4 * SL::kScrRow + n * 8 + 2 * t) =
                        make_float2(o[4 * c + n][0], o[4 * c + n][1]);
                    *reinterpret_cast<float2*>(my + (g4 + 8) * SL::kScrRow + n * 8 + 2 * t) =
                        make_float2(o[4 * c + n][2], o[4 * c + n][3]);
                }
                consumer_bar_sync();
                for (int idx = ctid; idx < rows * 32; idx += kCW * 32) {
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
                consumer_bar_sync();
            }
        }
    }
}

}  // namespace

size_t warp_kernel_smem_bytes(int head_dim) {
    return (head_dim == 128 ? SmemLayout<128>::kTotal : SmemLayout<64>::kTotal) + 1024;
}

cudaError_t configure_attention_kernels() {
    cudaError_t e = cudaFuncSetAttribute(seg_attn_warp_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)warp_kernel_smem_bytes(128));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(seg_attn_warp_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)warp_kernel_smem_bytes(64));
}

cudaError_t launch_seg_attn_warp(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnArgs& a,
                                 cudaStream_t stream) {
    if (a.grid == 0) return cudaSuccess;
    const size_t smem = warp_kernel_smem_bytes(a.head_dim);
    if (a.head_dim == 128)
        seg_attn_warp_kernel<128><<<a.grid, kThreads, smem, stream>>>(tm_k, tm_v, a);
    else
        seg_attn_warp_kernel<64><<<a.grid, kThreads, smem, stream>>>(tm_k, tm_v, a);
    return cudaGetLastError();
}

}  // namespace rksc
