// RSBCM eviction (Section 2.4, Algorithm 4): page scores from the attention's block masses, and
// the exact selection of the entries with the smallest omega = score / (depth + 1).
#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "kernels.h"
#include "rksc_internal.h"

namespace cg = cooperative_groups;

namespace rksc {
namespace {

constexpr int kScoreThreads = 256;
constexpr int kScoreWarps = kScoreThreads / 32;
constexpr int kScoreBatch = 32;        // sharers whose head sums are staged before they are added up

// One CTA per (segment, 32 consecutive pages): lane <-> page.  The warps share out the segment's
// sharers; each forms the head sum of its sharer (ascending h, fp64), and warp 0 then adds the
// head sums to the running score in ascending sharer order.  The order of every fp64 addition is
// thereby fixed: sum_b ( sum_h mass[b][h][j] ).
__global__ void __launch_bounds__(kScoreThreads) page_score_kernel(const int2* __restrict__ chunks,
                                                                   const int32_t* __restrict__ seg_block_off,
                                                                   const int32_t* __restrict__ seg_sharer_off,
                                                                   const Sharer* __restrict__ sharers,
                                                                   const float* __restrict__ mass,
                                                                   double* __restrict__ score, int Hq) {
    __shared__ double part[kScoreBatch][32];
    const int2 c = chunks[blockIdx.x];
    const int seg = c.x;
    const int lo = seg_block_off[seg];
    const int n = seg_block_off[seg + 1] - lo;
    const int sh0 = seg_sharer_off[seg];
    const int nsh = seg_sharer_off[seg + 1] - sh0;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int p = c.y + lane;
    const bool ok = p < n;
    double run = 0.0;
    for (int base = 0; base < nsh; base += kScoreBatch) {
        const int cnt = min(kScoreBatch, nsh - base);
        for (int i = warp; i < cnt; i += kScoreWarps) {
            const Sharer sh = sharers[sh0 + base + i];
            double hs = 0.0;
            if (ok) {
                const float* m = mass + sh.mass_base + p;
                const int64_t stride = sh.nblk;
#pragma unroll 8
                for (int h = 0; h < Hq; ++h) hs += (double)__ldg(m + h * stride);
            }
            part[i][lane] = hs;
        }
        __syncthreads();
        if (warp == 0)
            for (int i = 0; i < cnt; ++i) run += part[i][lane];
        __syncthreads();
    }
    if (warp == 0 && ok) score[lo + p] = run;
}

// omega as a 64-bit key whose unsigned order is the numeric order (zeros of either sign equal).
__device__ __forceinline__ uint64_t omega_key(double s, int32_t d) {
    double w = __ddiv_rn(s, (double)(d + 1));
    if (w == 0.0) w = 0.0;
    const uint64_t u = (uint64_t)__double_as_longlong(w);
    return (u >> 63) ? ~u : (u | (1ull << 63));
}

constexpr int kSelThreads = 1024;
constexpr int kSelWarps = kSelThreads / 32;
constexpr int kSelCluster = 8;          // CTAs of the one cluster that runs the selection

// Exact selection of the k entries smallest by (omega, index), by one thread-block cluster; CTA r
// owns the r-th contiguous slice of the entries.  A most-significant-byte-first radix select finds
// the k-th smallest key T and how many entries equal to T are still due: per pass every CTA
// histograms its slice, the cluster meets at its hardware barrier, and each CTA adds up all CTAs'
// histograms through distributed shared memory and takes the same decision.  A last sweep in
// index order marks key < T, and the first `due` entries with key == T.
__global__ void __launch_bounds__(kSelThreads) rsbcm_select_kernel(const double* __restrict__ score,
                                                                   const int32_t* __restrict__ depth, int32_t n,
                                                                   uint32_t k, uint64_t* __restrict__ keys,
                                                                   uint8_t* __restrict__ evicted,
                                                                   int32_t* __restrict__ num_evicted) {
    __shared__ uint32_t hist[kSelWarps][256];
    __shared__ uint32_t total[2][256];      // this CTA's histogram of the pass, read by the whole cluster
    __shared__ uint32_t gtotal[256];        // the cluster's histogram
    __shared__ uint64_t s_prefix;
    __shared__ uint32_t s_due, s_bin;
    __shared__ uint32_t warp_ties[kSelWarps];
    __shared__ uint32_t s_tie_base;
    cg::cluster_group cl = cg::this_cluster();
    const int rank = (int)cl.block_rank(), nrank = (int)cl.num_blocks();
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = (n + nrank - 1) / nrank;
    const int lo = min(n, rank * per), hi = min(n, lo + per);
    if (rank == 0 && tid == 0 && num_evicted) *num_evicted = (int32_t)k;
    if (k == 0 || k >= (uint32_t)n) {
        const uint8_t v = k == 0 ? 0 : 1;
        for (int i = lo + tid; i < hi; i += kSelThreads) evicted[i] = v;
        return;
    }
    for (int i = lo + tid; i < hi; i += kSelThreads) keys[i] = omega_key(score[i], depth[i]);
    if (tid == 0) {
        s_prefix = 0;
        s_due = k;
    }
    __syncthreads();
    for (int pass = 7; pass >= 0; --pass) {
        for (int i = tid; i < kSelWarps * 256; i += kSelThreads) (&hist[0][0])[i] = 0;
        __syncthreads();
        const uint64_t himask = pass == 7 ? 0ull : (~0ull << (8 * (pass + 1)));
        const uint64_t prefix = s_prefix;
        for (int i = lo + tid; i < hi; i += kSelThreads) {
            const uint64_t key = keys[i];
            if ((key & himask) == prefix) atomicAdd(&hist[warp][(key >> (8 * pass)) & 255], 1u);
        }
        __syncthreads();
        if (tid < 256) {
            uint32_t t = 0;
#pragma unroll
            for (int w = 0; w < kSelWarps; ++w) t += hist[w][tid];
            total[pass & 1][tid] = t;
        }
        // total[pass & 1] is next written two passes on, after another cluster barrier: no CTA can
        // still be reading it then.
        cl.sync();
        if (tid < 256) {
            uint32_t t = 0;
            for (int r = 0; r < nrank; ++r) t += *cl.map_shared_rank(&total[pass & 1][tid], r);
            gtotal[tid] = t;
        }
        __syncthreads();
        if (warp == 0) {
            // bin holding the due-th smallest candidate: lane l covers bins 8l .. 8l+7
            const uint32_t due = s_due;     // read by every lane before the shuffles below, written after them
            uint32_t mine = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) mine += gtotal[8 * lane + j];
            uint32_t incl = mine;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                const uint32_t v = __shfl_up_sync(0xffffffffu, incl, d);
                if (lane >= d) incl += v;
            }
            const uint32_t excl = incl - mine;
            if (excl < due && due <= incl) {
                uint32_t left = due - excl;
                int bin = 8 * lane;
                while (gtotal[bin] < left) left -= gtotal[bin++];
                s_due = left;
                s_bin = (uint32_t)bin;
                s_prefix = prefix | ((uint64_t)bin << (8 * pass));
            }
        }
        __syncthreads();
    }
    const uint64_t T = s_prefix;
    const uint32_t due = s_due;     // entries equal to T still to be marked, lowest indices first
    // entries equal to T in the slices before this one: the last pass's histograms hold them
    if (tid == 0) {
        uint32_t base = 0;
        for (int r = 0; r < rank; ++r) base += *cl.map_shared_rank(&total[0][s_bin], r);
        s_tie_base = base;
    }
    __syncthreads();
    for (int i0 = lo; i0 < hi; i0 += kSelThreads) {
        const int i = i0 + tid;
        const uint64_t key = i < hi ? keys[i] : ~0ull;
        const bool tie = i < hi && key == T;
        const uint32_t bal = __ballot_sync(0xffffffffu, tie);
        if (lane == 0) warp_ties[warp] = __popc(bal);
        __syncthreads();
        uint32_t before = s_tie_base;
        for (int w = 0; w < warp; ++w) before += warp_ties[w];
        before += __popc(bal & ((1u << lane) - 1u));
        if (i < hi) evicted[i] = (key < T || (tie && before < due)) ? 1 : 0;
        __syncthreads();
        if (tid == 0) {
            uint32_t t = s_tie_base;
            for (int w = 0; w < kSelWarps; ++w) t += warp_ties[w];
            s_tie_base = t;
        }
        __syncthreads();
    }
    cl.sync();      // no CTA leaves while another may still read its histogram
}

}  // namespace

cudaError_t launch_page_scores(const int2* chunks, int num_chunks, const int32_t* seg_block_off,
                               const int32_t* seg_sharer_off, const Sharer* sharers, const float* mass, double* score,
                               int Hq, cudaStream_t stream) {
    if (num_chunks <= 0) return cudaSuccess;
    page_score_kernel<<<num_chunks, kScoreThreads, 0, stream>>>(chunks, seg_block_off, seg_sharer_off, sharers, mass,
                                                                score, Hq);
    return cudaGetLastError();
}

cudaError_t launch_rsbcm_select(const double* score, const int32_t* depth, int32_t n, uint32_t k, uint64_t* keys,
                                uint8_t* evicted, int32_t* num_evicted, cudaStream_t stream) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3(kSelCluster);
    cfg.blockDim = dim3(kSelThreads);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = kSelCluster;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, rsbcm_select_kernel, score, depth, n, k, keys, evicted, num_evicted);
}

}  // namespace rksc

// ---- token-by-token decode: the new token's key and value into the paged pool ----
namespace rksc {
namespace {
// One warp per (branch, KV head): copies d bf16 of K and of V (16-byte pieces when d allows).
__global__ void kv_append_kernel(uint8_t* __restrict__ k_pool, uint8_t* __restrict__ v_pool, const uint8_t* __restrict__ k_new,
                                 const uint8_t* __restrict__ v_new, const int32_t* __restrict__ page,
                                 const int32_t* __restrict__ slot, int B, int Hkv, int row_bytes, int num_pool_blocks) {
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (gw >= B * Hkv) return;
    const int b = gw / Hkv, h = gw % Hkv;
    const int pg = page[b], sl = slot[b];
    if (pg < 0 || pg >= num_pool_blocks || sl < 0 || sl >= kBlock) return;   // no token for this branch (or a bad entry: skipped)
    const size_t dst = (((size_t)pg * Hkv + h) * kBlock + sl) * row_bytes;
    const size_t src = ((size_t)b * Hkv + h) * row_bytes;
    if ((row_bytes & 15) == 0) {
        for (int i = lane * 16; i < row_bytes; i += 32 * 16) {
            *reinterpret_cast<uint4*>(k_pool + dst + i) = *reinterpret_cast<const uint4*>(k_new + src + i);
            *reinterpret_cast<uint4*>(v_pool + dst + i) = *reinterpret_cast<const uint4*>(v_new + src + i);
        }
    } else {
        for (int i = lane * 2; i < row_bytes; i += 64) {
            *reinterpret_cast<uint16_t*>(k_pool + dst + i) = *reinterpret_cast<const uint16_t*>(k_new + src + i);
            *reinterpret_cast<uint16_t*>(v_pool + dst + i) = *reinterpret_cast<const uint16_t*>(v_new + src + i);
        }
    }
}
}  // namespace

cudaError_t launch_kv_append(void* k_pool, void* v_pool, const void* k_new, const void* v_new, const int32_t* page,
                             const int32_t* slot, int B, int Hkv, int head_dim, int num_pool_blocks, cudaStream_t stream) {
    if (B <= 0) return cudaSuccess;
    const int warps = B * Hkv;
    kv_append_kernel<<<(warps + 7) / 8, 256, 0, stream>>>(static_cast<uint8_t*>(k_pool), static_cast<uint8_t*>(v_pool),
                                                         static_cast<const uint8_t*>(k_new), static_cast<const uint8_t*>(v_new),
                                                         page, slot, B, Hkv, head_dim * 2, num_pool_blocks);
    return cudaGetLastError();
}
}  // namespace rksc
