// Log-sum-exp merge of the partial results of one (branch, query head), and the final
// normalisation of the per-block softmax masses.
//
// The segment kernels leave, for every (segment chunk, row), a normalised partial output and its
// log2-sum-exp, and in block_mass the log2 of every page's unnormalised mass.  Here:
//   LSE  = log2 sum_p 2^lse_p
//   out  = sum_p 2^(lse_p - LSE) * O_p
//   mass_j = 2^(logmass_j - LSE)
// which is exactly softmax attention over the concatenation of the branch's segments.
#include "kernels.h"

namespace rksc {

namespace {

constexpr int kMergeThreads = 128;

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm volatile("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__global__ void __launch_bounds__(kMergeThreads)
merge_kernel(const AttnArgs a) {
    const int bh = blockIdx.x;
    const int b = bh / a.Hq, h = bh % a.Hq;
    const int kvh = h / a.G, gi = h % a.G;
    const int HD = a.head_dim;
    const int lo = a.plan.merge_off[b * a.Hkv + kvh], hi = a.plan.merge_off[b * a.Hkv + kvh + 1];
    const int tid = threadIdx.x;
    __shared__ float red[kMergeThreads / 32];
    __shared__ float s_lse;

    // max and sum of the parts' log2-sum-exp (block reduction; the list is short)
    float mx = -INFINITY;
    for (int i = lo + tid; i < hi; i += kMergeThreads) mx = fmaxf(mx, a.part_lse[a.plan.merge_rows[i] + gi]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if ((tid & 31) == 0) red[tid >> 5] = mx;
    __syncthreads();
    mx = fmaxf(fmaxf(red[0], red[1]), fmaxf(red[2], red[3]));
    __syncthreads();
    float sum = 0.f;
    for (int i = lo + tid; i < hi; i += kMergeThreads) sum += fast_exp2(a.part_lse[a.plan.merge_rows[i] + gi] - mx);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
    if ((tid & 31) == 0) red[tid >> 5] = sum;
    __syncthreads();
    if (tid == 0) s_lse = mx + log2f((red[0] + red[1]) + (red[2] + red[3]));
    __syncthreads();
    const float lse = s_lse;

    float* out = a.out + (size_t)bh * HD;
    if (hi == lo) {   // the branch attends to nothing
        for (int c = tid; c < HD; c += kMergeThreads) out[c] = 0.f;
        return;
    }
    for (int c = tid; c < HD; c += kMergeThreads) {
        float acc = 0.f;
        for (int i = lo; i < hi; ++i) {
            const int row = a.plan.merge_rows[i] + gi;
            acc += fast_exp2(a.part_lse[row] - lse) * a.part_o[(size_t)row * HD + c];
        }
        out[c] = acc;
    }
    if (a.block_mass != nullptr) {
        const int nblk = a.plan.br_nblk[b];
        float* mass = a.block_mass + a.plan.mass_off[b] * a.Hq + (int64_t)h * nblk;
        for (int j = tid; j < nblk; j += kMergeThreads) mass[j] = fast_exp2(mass[j] - lse);
    }
}

}  // namespace

cudaError_t launch_merge(const AttnArgs& a, cudaStream_t stream) {
    const int n = a.B * a.Hq;
    if (n == 0) return cudaSuccess;
    merge_kernel<<<n, kMergeThreads, 0, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace rksc
