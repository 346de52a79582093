// Segment attention for work items with at most 8 stacked rows (a private suffix or prefix copy:
// R = G query heads of one branch on one KV head) - the bulk of the bytes in batched serving.
//
// Every WARP is an independent worker: it claims items (at most 32 pages each) from a global
// counter, streams their pages through a private ring of page slots by TMA (cp.async.bulk.tensor,
// 128-byte swizzle, no multicast; one box per 4 KiB K or V tile), and re-issues a slot itself as soon as
// it has read it - so no other warp stands between a landed page and the next copy, which is what
// keeps enough bytes in flight to approach the HBM rate.  The next item is claimed one ahead and
// its first pages are requested while the current item's last pages are processed.
//
// Per page (16 tokens): S^T = K Q^T (mma.sync m16n8k16: M = 16 tokens, N = 8 rows, bf16 in, fp32
// out), online softmax in base 2 over the token dimension (shuffles across the 8 row groups),
// the page's softmax mass as log2 to block_mass, P^T split into bf16 high + low parts and moved to
// the B-operand layout with movmatrix, O^T += V^T P^T.  O^T is rescaled only when a running
// maximum moved.  At the end of an item the warp writes its rows' normalised partial output and
// log2-sum-exp to the workspace (no merge inside the CTA: the warp saw every page of the item).
// Every wait is bounded; on expiry the warp records RKSC_ERR_DEVICE_TIMEOUT and stops.
#include <cuda_bf16.h>

#include "kernels.h"

namespace rksc {

namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kR = 2;   // page slots per warp

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
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
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t x) {
    uint32_t y;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(y) : "r"(x));
    return y;
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
__device__ __forceinline__ void split_pack(float a, float b, uint32_t& hi, uint32_t& lo) {
    const __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    const float2 hf = __bfloat1622float2(h);
    const __nv_bfloat162 l = __floats2bfloat162_rn(a - hf.x, b - hf.y);
    hi = *reinterpret_cast<const uint32_t*>(&h);
    lo = *reinterpret_cast<const uint32_t*>(&l);
}

template <int HD>
__global__ void __launch_bounds__(kThreads, 2)
seg_attn_small_kernel(const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v,
                      const AttnArgs a) {
    constexpr int KS = HD / 16;
    constexpr int kTile = kBlock * HD * 2;     // K (or V) of one page
    constexpr int kPage = 2 * kTile;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t ring = smem_u32(smem) + warp * (kR * kPage);
    const uint32_t bars = smem_u32(smem) + kWarps * kR * kPage + warp * (kR * 8);

    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (lane == 0) {
        for (int i = 0; i < kR; ++i) mbar_init(bars + 8 * i, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();

    const int first_item = a.num_tc_items, end_item = a.num_tc_items + a.num_small_items;
    auto claim = [&]() {
        int v = 0;
        if (lane == 0) v = first_item + atomicAdd(a.counters + 4, 1);
        return __shfl_sync(0xffffffffu, v, 0);
    };
    auto fetch_item = [&](int i) {
        WorkItem w{};
        if (i < end_item) w = a.plan.items[i];
        return w;
    };
    auto fetch_ids = [&](const WorkItem& w) {   // an item of this class has at most 32 pages: one id per lane
        return (lane < w.num_pages) ? __ldg(a.plan.seg_blocks + w.page_begin + lane) : 0;
    };
    // stage page `p` of item (w, ids) into ring slot `seq % kR`
    auto issue = [&](const WorkItem& w, int ids, int p, int seq) {
        const int page = __shfl_sync(0xffffffffu, ids, p);
        const int slot = seq % kR;
        const uint32_t bar = bars + 8 * slot;
        if (lane == 0) mbar_arrive_expect_tx(bar, kPage);
        __syncwarp();
        if (lane < 2) {
            // The tile (16 tokens x HD) is fetched as kRowsPerTok x 16 rows of 64 elements: shared-memory
            // row 2*tok + half holds dims [64*half, 64*half + 64) of the token, 16-byte chunks swizzled
            // by the row index (one TMA request per tile instead of one per half).
            const int y = (page * a.Hkv + w.kv_head) * (kBlock * (HD / 64));
            tma_load_2d(ring + slot * kPage + lane * kTile, lane ? &tm_v : &tm_k, 0, y, bar);
        }
    };

    const int g4 = lane >> 2, t = lane & 3;
    const int a_tok = ((lane >> 4) << 3) + (lane & 7), a_chunk = (lane >> 3) & 1;
    const int b_tok = (((lane >> 3) & 1) << 3) + (lane & 7), b_chunk = lane >> 4;
    // byte offset of 16-byte chunk c16 (of HD/8) of token `tok` inside a staged tile
    auto tile_addr = [](int tok, int c16) -> uint32_t {
        if (HD == 128) {
            const int row = 2 * tok + (c16 >> 3);
            return (uint32_t)(row * 128 + (((c16 & 7) ^ (row & 7)) << 4));
        }
        return (uint32_t)(tok * 128 + ((c16 ^ (tok & 7)) << 4));
    };
    const float scale_log2 = a.scale_log2;
    const int G = a.G;

    int idx = claim();
    WorkItem it = fetch_item(idx);
    int ids = fetch_ids(it);
    int seq_i = 0, seq_c = 0;     // pages issued / consumed by this warp so far
    int iss_cur = 0;              // pages of the current item already issued
    bool ok = true;

    while (idx < end_item && ok) {
        // the item after this one: claimed now, its first pages are requested as this one drains
        const int nidx = claim();
        const WorkItem nit = fetch_item(nidx);
        const int nids = fetch_ids(nit);
        int iss_nxt = 0;
        while (seq_i - seq_c < kR && iss_cur < it.num_pages) issue(it, ids, iss_cur++, seq_i++);

        // ---- rows and queries of this item: thread rows 2t, 2t+1 (softmax), query of row g4 (B operand) ----
        const int rows = it.num_sharers * G;   // <= 8
        const int r0 = 2 * t, r1 = 2 * t + 1;
        const bool v0 = r0 < rows, v1 = r1 < rows;
        int64_t mb0 = 0, mb1 = 0;
        if (v0) {
            const Sharer sh = a.plan.sharers[it.sharer_begin + r0 / G];
            mb0 = sh.mass_base + (int64_t)(it.kv_head * G + r0 % G) * sh.nblk + it.seg_page_begin;
        }
        if (v1) {
            const Sharer sh = a.plan.sharers[it.sharer_begin + r1 / G];
            mb1 = sh.mass_base + (int64_t)(it.kv_head * G + r1 % G) * sh.nblk + it.seg_page_begin;
        }
        uint32_t qf[KS][2];
        {
            const bool qv = g4 < rows;
            const uint32_t* q0 = nullptr;
            if (qv) {
                const int br = a.plan.sharers[it.sharer_begin + g4 / G].branch;
                q0 = reinterpret_cast<const uint32_t*>(a.q) + ((size_t)br * a.Hq + it.kv_head * G + g4 % G) * (HD / 2);
            }
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                qf[ks][0] = qv ? __ldg(q0 + ks * 8 + t) : 0u;
                qf[ks][1] = qv ? __ldg(q0 + ks * 8 + 4 + t) : 0u;
            }
        }
        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[2 * KS][4];   // O^T: high parts of P in [0, KS), low parts in [KS, 2 KS)
#pragma unroll
        for (int n = 0; n < 2 * KS; ++n) o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f;

        for (int pi = 0; pi < it.num_pages; ++pi, ++seq_c) {
            const int slot = seq_c % kR;
            ok = mbar_wait(bars + 8 * slot, (uint32_t)(seq_c / kR) & 1u);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            const uint32_t kb = ring + slot * kPage, vb = kb + kTile;
            const int nv = it.num_tokens - pi * kBlock;   // valid tokens of the page: >= 1, >= 16 if full
#ifdef RKSC_SKIP_COMPUTE
            if (nv > -1000) {
                __syncwarp();
                if (iss_cur < it.num_pages) issue(it, ids, iss_cur++, seq_i++);
                else if (nidx < end_item && iss_nxt < nit.num_pages) issue(nit, nids, iss_nxt++, seq_i++);
                continue;
            }
#endif

            // S^T = K Q^T: 16 tokens x 8 rows; thread: tokens g4, g4+8; rows 2t, 2t+1
            float s[4] = {0.f, 0.f, 0.f, 0.f}, s_odd[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t ak[4];
                ldmatrix_x4(kb + tile_addr(b_tok, ks * 2 + b_chunk), ak);
                if (ks & 1) mma_bf16(s_odd, ak, qf[ks][0], qf[ks][1]);
                else mma_bf16(s, ak, qf[ks][0], qf[ks][1]);
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
                // log2 of the page's unnormalised mass, absolute (not relative to the running max)
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
#pragma unroll
            for (int n = 0; n < KS; ++n) {
                uint32_t av[4];
                ldmatrix_x4_trans(vb + tile_addr(a_tok, n * 2 + a_chunk), av);
                mma_bf16(o[n], av, bh0, bh1);
                mma_bf16(o[KS + n], av, bl0, bl1);
            }
            // the slot has been read: request the next page into it (this item's, else the next item's)
            __syncwarp();
            if (iss_cur < it.num_pages) issue(it, ids, iss_cur++, seq_i++);
            else if (nidx < end_item && iss_nxt < nit.num_pages) issue(nit, nids, iss_nxt++, seq_i++);
        }
        if (!ok) break;

        // ---- partial result of the item: normalised O and log2-sum-exp per row ----
        {
            const float i0 = 1.f / l0, i1 = 1.f / l1;
            float* d0 = a.part_o + ((size_t)it.part_row_base + r0) * HD;
            float* d1 = a.part_o + ((size_t)it.part_row_base + r1) * HD;
#pragma unroll
            for (int n = 0; n < KS; ++n) {
                if (v0) {
                    d0[n * 16 + g4] = (o[n][0] + o[KS + n][0]) * i0;
                    d0[n * 16 + g4 + 8] = (o[n][2] + o[KS + n][2]) * i0;
                }
                if (v1) {
                    d1[n * 16 + g4] = (o[n][1] + o[KS + n][1]) * i1;
                    d1[n * 16 + g4 + 8] = (o[n][3] + o[KS + n][3]) * i1;
                }
            }
            if (g4 == 0) {
                if (v0) a.part_lse[it.part_row_base + r0] = m0 + fast_log2(l0);
                if (v1) a.part_lse[it.part_row_base + r1] = m1 + fast_log2(l1);
            }
        }
        idx = nidx;
        it = nit;
        ids = nids;
        iss_cur = iss_nxt;
    }
    if (!ok && lane == 0 && a.status) atomicExch(a.status, RKSC_ERR_DEVICE_TIMEOUT);

    // the last warp of the grid to stop claiming rewinds the counters for the next launch
    if (lane == 0) {
        __threadfence();
        const int done = atomicAdd(a.counters + 5, 1);
        if (done == (int)(gridDim.x * kWarps) - 1) {
            a.counters[4] = 0;
            a.counters[5] = 0;
            __threadfence();
        }
    }
    // launched behind another segment kernel without waiting for it: do not complete before it has
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

}  // namespace

size_t small_kernel_smem_bytes(int head_dim) {
    return (size_t)kWarps * kR * (2 * kBlock * head_dim * 2) + kWarps * kR * 8 + 1024;
}

cudaError_t configure_small_kernel() {
    cudaError_t e = cudaFuncSetAttribute(seg_attn_small_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)small_kernel_smem_bytes(128));
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(seg_attn_small_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)small_kernel_smem_bytes(64));
}

cudaError_t launch_seg_attn_small(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnArgs& a,
                                  cudaStream_t stream, bool chained) {
    if (a.grid_small == 0) return cudaSuccess;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.grid_small, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = small_kernel_smem_bytes(a.head_dim);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = chained ? 1 : 0;
    if (a.head_dim == 128) return cudaLaunchKernelEx(&cfg, seg_attn_small_kernel<128>, tm_k, tm_v, a);
    return cudaLaunchKernelEx(&cfg, seg_attn_small_kernel<64>, tm_k, tm_v, a);
}

}  // namespace rksc
