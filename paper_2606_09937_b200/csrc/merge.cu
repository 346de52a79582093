// Log-sum-exp merge of the partial results of one (branch, query head), and the final
// normalisation of the per-block softmax masses.
//
// The segment kernel leaves, for every (segment chunk, row), a normalised partial output and its
// log2-sum-exp, and in block_mass the log2 of every page's unnormalised mass.  Here:
//   LSE  = log2 sum_p 2^lse_p
//   out  = sum_p 2^(lse_p - LSE) * O_p
//   mass_j = 2^(logmass_j - LSE)
// which is exactly softmax attention over the concatenation of the branch's segments.
//
// One warp (or, when there are few (branch, head) pairs, 2/4/8 warps) per (branch, head): lanes split
// the head dimension four columns each (16-byte loads of the partial rows) and stride over the parts;
// the warps of a pair each recompute the (cheap) LSE and share out the pair's blocks, so that the
// mass pass has enough loads in flight even when B x Hq is small and the context is long.  The kernel is launched with
// programmatic stream serialisation: its blocks may become resident while the segment kernel
// drains, read their (plan-owned) part lists, and then wait for the segment kernel's results.
#include "kernels.h"

namespace rksc {

namespace {

constexpr int kMergeWarps = 8;
constexpr int kMergeThreads = kMergeWarps * 32;

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

constexpr int kPartBatch = 8;   // partial rows a lane has in flight at once
constexpr int kMassBatch = 8;   // block masses a lane has in flight at once

__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const AttnArgs a, const int wpk_log2) {
    const int lane = threadIdx.x & 31;
    const int gw = blockIdx.x * (int)(blockDim.x >> 5) + (threadIdx.x >> 5);   // global warp
    const int bh = gw >> wpk_log2;
    const int sub = gw & ((1 << wpk_log2) - 1), wpk = 1 << wpk_log2;
    const bool live = bh < a.B * a.Hq;
    int b = 0, h = 0, lo = 0, hi = 0, nblk = 0;
    float* mass = nullptr;
    if (live) {
        b = bh / a.Hq;
        h = bh % a.Hq;
        const int key = b * a.Hkv + h / a.G;
        lo = a.plan.merge_off[key];
        hi = a.plan.merge_off[key + 1];
        if (a.block_mass != nullptr && hi > lo) {
            nblk = a.plan.br_nblk[b];
            mass = a.block_mass + a.plan.mass_off[b] * a.Hq + (int64_t)h * nblk;
        }
    }
    const int gi = h % a.G;
    const int HD = a.head_dim;
    // the first 32 part rows of this warp's list (plan data: readable before the dependency resolves)
    const int row_l = (lo + lane < hi) ? a.plan.merge_rows[lo + lane] + gi : -1;

    // a kernel launched behind this one with programmatic serialisation may set itself up meanwhile
    // (it waits for this grid's completion before it touches memory)
    if (threadIdx.x == 0) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    // everything below reads what the segment kernel wrote
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (!live) return;

    // Everything this warp needs is fetched with as few dependent round trips to L2 as possible: the
    // log-sum-exps of the parts, the first batch of partial rows and the first batch of block masses
    // are all requested before anything is reduced.
    const bool has_cols = (4 * lane < HD) && sub == 0;
    const float my_lse = (row_l >= 0) ? a.part_lse[row_l] : -INFINITY;
    const int n0 = min(32, hi - lo);
    float4 v[kPartBatch];
#pragma unroll
    for (int j = 0; j < kPartBatch; ++j) {
        const int row = __shfl_sync(0xffffffffu, row_l, j);
        v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (has_cols && j < n0) v[j] = *reinterpret_cast<const float4*>(a.part_o + (size_t)row * HD + 4 * lane);
    }
    const int stride = 32 * wpk;
    float mv[kMassBatch];
#pragma unroll
    for (int k = 0; k < kMassBatch; ++k) {
        const int j = sub * 32 + lane + k * stride;
        mv[k] = (j < nblk) ? mass[j] : 0.f;
    }

    // LSE over the parts
    float mx = my_lse;
    for (int i = lo + 32 + lane; i < hi; i += 32) mx = fmaxf(mx, a.part_lse[a.plan.merge_rows[i] + gi]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    float sum = (row_l >= 0) ? fast_exp2(my_lse - mx) : 0.f;
    for (int i = lo + 32 + lane; i < hi; i += 32) sum += fast_exp2(a.part_lse[a.plan.merge_rows[i] + gi] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    const float lse = mx + log2f(sum);

    // out (first warp of the pair): lane owns columns 4*lane .. 4*lane+3
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (sub == 0) {
        for (int i0 = lo; i0 < hi; i0 += 32) {
            const int n = min(32, hi - i0);
            const int my_row = (i0 == lo) ? row_l : ((i0 + lane < hi) ? a.plan.merge_rows[i0 + lane] + gi : -1);
            const float my_w = (my_row < 0) ? 0.f : fast_exp2(((i0 == lo) ? my_lse : a.part_lse[my_row]) - lse);
            for (int j0 = 0; j0 < n; j0 += kPartBatch) {
                if (i0 != lo || j0 != 0) {   // the very first batch is already here
#pragma unroll
                    for (int j = 0; j < kPartBatch; ++j) {
                        const int row = __shfl_sync(0xffffffffu, my_row, (j0 + j) & 31);
                        v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
                        if (has_cols && j0 + j < n)
                            v[j] = *reinterpret_cast<const float4*>(a.part_o + (size_t)row * HD + 4 * lane);
                    }
                }
#pragma unroll
                for (int j = 0; j < kPartBatch; ++j) {
                    const float w = __shfl_sync(0xffffffffu, my_w, (j0 + j) & 31);   // 0 past the end of the list
                    const float wj = (j0 + j < n) ? w : 0.f;
                    acc.x += wj * v[j].x;
                    acc.y += wj * v[j].y;
                    acc.z += wj * v[j].z;
                    acc.w += wj * v[j].w;
                }
            }
        }
    }
    if (has_cols) *reinterpret_cast<float4*>(a.out + (size_t)bh * HD + 4 * lane) = acc;   // zeros when there are no parts

    // block masses: mass_j = 2^(logmass_j - LSE), in place
    for (int j0 = sub * 32 + lane; j0 < nblk; j0 += kMassBatch * stride) {
        if (j0 != sub * 32 + lane) {
#pragma unroll
            for (int k = 0; k < kMassBatch; ++k) {
                const int j = j0 + k * stride;
                mv[k] = (j < nblk) ? mass[j] : 0.f;
            }
        }
#pragma unroll
        for (int k = 0; k < kMassBatch; ++k) {
            const int j = j0 + k * stride;
            if (j < nblk) mass[j] = fast_exp2(mv[k] - lse);
        }
    }
}

}  // namespace

cudaError_t launch_merge(const AttnArgs& a, cudaStream_t stream, bool early_residency) {
    const int n = a.B * a.Hq;
    if (n == 0) return cudaSuccess;
    int wpk_log2 = 0;   // warps per (branch, head): enough warps to fill the device
    while (wpk_log2 < 3 && ((int64_t)n << (wpk_log2 + 1)) <= 8192) ++wpk_log2;
    const int64_t warps = (int64_t)n << wpk_log2;
    // Eight warps per block when eight warps share a (branch, head) - they then sit in one block and
    // share its cache lines (split over two blocks: 58 -> 72 us per call on the long-context
    // configuration) - and four otherwise: the smaller blocks find room on an SM sooner as the segment
    // kernel's CTAs leave (measured: 0.3-1.5 us per call on batched serving and Tree-of-Thoughts).
    const int block_warps = wpk_log2 == 3 ? kMergeWarps : kMergeWarps / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((warps + block_warps - 1) / block_warps), 1, 1);
    cfg.blockDim = dim3(block_warps * 32, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = early_residency ? 1 : 0;   // without the attribute the merge starts when the segment kernel has completed
    return cudaLaunchKernelEx(&cfg, merge_kernel, a, wpk_log2);
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded wait (rksc_debug_wait_timeout): same structure as the kernels' waits -
// try_wait with a suspend hint in a loop, the SM cycle counter as the limit, an abort flag in shared
// memory that makes every later wait of the CTA return at once, the status word written once.
// ---------------------------------------------------------------------------------------------
namespace {

__global__ void __launch_bounds__(128) wait_timeout_kernel(long long limit, int32_t* status) {
    __shared__ __align__(8) unsigned long long bar;
    __shared__ int abort_flag;
    const uint32_t b = static_cast<uint32_t>(__cvta_generic_to_shared(&bar));
    if (threadIdx.x == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(b) : "memory");   // one arrival expected, none comes
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    for (int round = 0; round < 3; ++round) {     // after the first expiry the later waits return at once
        if (*reinterpret_cast<volatile int*>(&abort_flag)) break;
        const long long t0 = clock64();
        for (;;) {
            uint32_t ok;
            asm volatile(
                "{\n"
                ".reg .pred p;\n"
                "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n"
                "selp.u32 %0, 1, 0, p;\n"
                "}\n"
                : "=r"(ok)
                : "r"(b), "r"(0u), "r"(1000u)
                : "memory");
            if (ok) break;
            if (clock64() - t0 > limit) {
                abort_flag = 1;
                if (status) atomicExch(status, RKSC_ERR_DEVICE_TIMEOUT);
                break;
            }
        }
    }
}

}  // namespace

cudaError_t launch_wait_timeout(long long limit, int32_t* status, cudaStream_t stream) {
    wait_timeout_kernel<<<1, 128, 0, stream>>>(limit, status);
    return cudaGetLastError();
}

}  // namespace rksc
