// Launch prototypes of the kernels (implemented in the .cu files of this directory).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>

#include "rksc_internal.h"

namespace rksc {

cudaError_t launch_asks_gate(const float* h_branch, const float* h_root, const int32_t* cand_prefix,
                             int B, int P, int L, int D, float alpha, float tau,
                             int32_t* branch_to_prefix, float* sigma, cudaStream_t stream);

struct AttnArgs {
    DevicePlan plan;
    const void* q;          // bf16 [B][Hq][d]
    float* part_o;          // [rows][d]
    float* part_lse;        // [rows], log2 units
    float* block_mass;      // may be null; holds log2 masses between the two launches
    float* out;             // [B][Hq][d]
    int32_t* status;        // may be null
    int32_t* counters;      // [2]: next work item, CTAs done; zero between launches
    int num_items;
    int num_tc_items;       // items [0, num_tc_items) go to the tcgen05 kernel, the rest to the warp kernel
    int grid_warp, grid_tc; // persistent CTAs of the two segment kernels
    int B, Hq, Hkv, G, head_dim;
    float scale_log2;       // sm_scale * log2(e)
};

// Sets the kernels' shared-memory attribute for the current device.
cudaError_t configure_attention_kernels();
size_t warp_kernel_smem_bytes(int head_dim);

size_t tc_kernel_smem_bytes();

// after_tc: the tcgen05 kernel was launched just before on the same stream; the warp kernel then
// starts as that one drains (programmatic dependent launch) and waits for it before it exits.
cudaError_t launch_seg_attn_warp(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnArgs& a,
                                 cudaStream_t stream, bool after_tc);
cudaError_t launch_seg_attn_tc(const CUtensorMap& tm_k, const CUtensorMap& tm_v, const AttnArgs& a,
                               cudaStream_t stream);
cudaError_t launch_merge(const AttnArgs& a, cudaStream_t stream, bool early_residency);

// RSBCM (Section 2.4, Algorithm 4): per-entry scores from the block masses; exact selection of the
// k entries smallest by (score / (depth + 1), index).  keys: scratch of n 64-bit words.
cudaError_t launch_page_scores(const int2* chunks, int num_chunks, const int32_t* seg_block_off,
                               const int32_t* seg_sharer_off, const Sharer* sharers, const float* mass, double* score,
                               int Hq, cudaStream_t stream);
// CGEE numerics (Section 2.3): entropy and top-1 probability of softmax(h W_u^T) for up to
// cgee_rows_per_launch() rows of h; exit test; verify-skip gate.
size_t cgee_smem_bytes(int D, int B);
int cgee_rows_per_launch();
cudaError_t configure_cgee_kernel(int max_smem);
cudaError_t launch_logit_entropy(const CUtensorMap& tm_w, const CUtensorMap& tm_h, int B, int D, long long V, int grid,
                                 float* partial, float* entropy, float* top1, int32_t* status, cudaStream_t stream);
cudaError_t launch_entropy_exit(const float* H, const float* H_prev, int B, int layer, int l_min, float theta, float eps,
                                int32_t* flags, cudaStream_t stream);
cudaError_t launch_verify_skip(const float* top1_steps, int t, int B, float tau_conf, float r_gap, float* p_out,
                               int32_t* skip, cudaStream_t stream);
cudaError_t launch_kv_append(void* k_pool, void* v_pool, const void* k_new, const void* v_new, const int32_t* page,
                             const int32_t* slot, int B, int Hkv, int head_dim, int num_pool_blocks, cudaStream_t stream);
cudaError_t launch_rsbcm_select(const double* score, const int32_t* depth, int32_t n, uint32_t k, uint64_t* keys,
                                uint8_t* evicted, int32_t* num_evicted, cudaStream_t stream);

cudaError_t launch_wait_timeout(long long limit_cycles, int32_t* status, cudaStream_t stream);

}  // namespace rksc
