// ASKS similarity gate (paper Eq. 2, Algorithm 2) as one launch.
//
// One thread-block cluster (up to 4 CTAs of 8 warps) per branch.  Every warp of the cluster takes whole layers: it
// streams the branch's and the candidate root's D-vector of that layer once with 16-byte
// loads, reduces dot / |h_b|^2 / |h_r|^2 with warp shuffles, and accumulates
// exp(alpha*(l-L)/L) * cos_l and exp(alpha*(l-L)/L) (the factor exp(-alpha) cancels in the
// ratio, which keeps the exponent <= 0).  The per-CTA sums meet in the shared memory of the
// cluster's first CTA (distributed shared memory), which forms sigma and the decision.  No
// scratch memory, no atomics, a fixed summation order.
#include <cooperative_groups.h>
#include <cuda_runtime.h>

#include "kernels.h"

namespace cg = cooperative_groups;

namespace rksc {

namespace {

constexpr int kGateWarps = 8;
constexpr int kGateThreads = kGateWarps * 32;
constexpr int kMaxCluster = 4;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

template <bool VEC4>
__device__ __forceinline__ void layer_sums(const float* __restrict__ hb, const float* __restrict__ hr,
                                           int D, int lane, float& dot, float& nb, float& nr) {
    dot = nb = nr = 0.f;
    if (VEC4) {
        const float4* b4 = reinterpret_cast<const float4*>(hb);
        const float4* r4 = reinterpret_cast<const float4*>(hr);
        const int n4 = D >> 2;
        int i = lane;
        for (; i + 96 < n4; i += 128) {   // 4 x 2 independent 16-byte loads in flight per lane
            float4 x[4], y[4];
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                x[u] = __ldcs(b4 + i + 32 * u);   // branch vectors are read once: streaming
                y[u] = __ldg(r4 + i + 32 * u);    // roots are re-read by every branch of the problem
            }
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                dot += x[u].x * y[u].x + x[u].y * y[u].y + x[u].z * y[u].z + x[u].w * y[u].w;
                nb += x[u].x * x[u].x + x[u].y * x[u].y + x[u].z * x[u].z + x[u].w * x[u].w;
                nr += y[u].x * y[u].x + y[u].y * y[u].y + y[u].z * y[u].z + y[u].w * y[u].w;
            }
        }
        for (; i < n4; i += 32) {
            const float4 x = __ldcs(b4 + i), y = __ldg(r4 + i);
            dot += x.x * y.x + x.y * y.y + x.z * y.z + x.w * y.w;
            nb += x.x * x.x + x.y * x.y + x.z * x.z + x.w * x.w;
            nr += y.x * y.x + y.y * y.y + y.z * y.z + y.w * y.w;
        }
    } else {
        for (int i = lane; i < D; i += 32) {
            const float x = hb[i], y = hr[i];
            dot += x * y;
            nb += x * x;
            nr += y * y;
        }
    }
    dot = warp_sum(dot);
    nb = warp_sum(nb);
    nr = warp_sum(nr);
}

template <bool VEC4>
__global__ void __launch_bounds__(kGateThreads)
asks_gate_kernel(const float* __restrict__ h_branch, const float* __restrict__ h_root,
                 const int32_t* __restrict__ cand_prefix, int B, int P, int L, int D,
                 float alpha, float tau, int32_t* __restrict__ branch_to_prefix,
                 float* __restrict__ sigma) {
    cg::cluster_group cluster = cg::this_cluster();
    const int csize = (int)cluster.num_blocks();
    const int crank = (int)cluster.block_rank();
    const int b = blockIdx.x / csize;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    __shared__ float warp_part[kGateWarps][2];
    __shared__ float cta_part[kMaxCluster][2];   // filled in the cluster's first CTA only

    const int r = cand_prefix[b];
    const bool r_ok = (r >= 0 && r < P);
    float num = 0.f, den = 0.f;
    if (r_ok) {
        const float* hb = h_branch + (size_t)b * L * D;
        const float* hr = h_root + (size_t)r * L * D;
        for (int l = crank * kGateWarps + warp; l < L; l += csize * kGateWarps) {
            float dot, nb, nr;
            layer_sums<VEC4>(hb + (size_t)l * D, hr + (size_t)l * D, D, lane, dot, nb, nr);
            // zero norm: the layer contributes 0; NaN flows through to sigma
            const float c = (nb == 0.f || nr == 0.f) ? 0.f : dot / (sqrtf(nb) * sqrtf(nr));
            const float e = expf(alpha * (float)(l + 1 - L) / (float)L);
            num += e * c;
            den += e;
        }
    }
    if (lane == 0) {
        warp_part[warp][0] = num;
        warp_part[warp][1] = den;
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        float n = 0.f, d = 0.f;
#pragma unroll
        for (int w = 0; w < kGateWarps; ++w) {
            n += warp_part[w][0];
            d += warp_part[w][1];
        }
        float* dst = cluster.map_shared_rank(&cta_part[0][0], 0);
        dst[2 * crank + 0] = n;
        dst[2 * crank + 1] = d;
    }
    cluster.sync();
    if (crank == 0 && threadIdx.x == 0) {
        float n = 0.f, d = 0.f;
        for (int c = 0; c < csize; ++c) {
            n += cta_part[c][0];
            d += cta_part[c][1];
        }
        const float s = r_ok ? n / d : __int_as_float(0x7fc00000);
        if (sigma) sigma[b] = s;
        branch_to_prefix[b] = (s >= tau) ? r : -1;
    }
}

}  // namespace

cudaError_t launch_asks_gate(const float* h_branch, const float* h_root, const int32_t* cand_prefix,
                             int B, int P, int L, int D, float alpha, float tau,
                             int32_t* branch_to_prefix, float* sigma, cudaStream_t stream) {
    // cluster size: enough warps to give every layer its own warp, at most kMaxCluster CTAs (larger
    // clusters of smaller CTAs were measured to limit how many clusters the device keeps resident)
    int csize = 1;
    while (csize < kMaxCluster && csize * kGateWarps < L) csize <<= 1;
    const bool vec4 = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(h_branch) & 15) == 0) &&
                      ((reinterpret_cast<uintptr_t>(h_root) & 15) == 0);

    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)((size_t)B * csize), 1, 1);
    cfg.blockDim = dim3(kGateThreads, 1, 1);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = csize;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    if (vec4)
        return cudaLaunchKernelEx(&cfg, asks_gate_kernel<true>, h_branch, h_root, cand_prefix, B, P, L, D,
                                  alpha, tau, branch_to_prefix, sigma);
    return cudaLaunchKernelEx(&cfg, asks_gate_kernel<false>, h_branch, h_root, cand_prefix, B, P, L, D,
                              alpha, tau, branch_to_prefix, sigma);
}

}  // namespace rksc
