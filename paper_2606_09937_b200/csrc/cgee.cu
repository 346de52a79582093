// CGEE numerics (Section 2.3): the entropy and top-1 probability of softmax(h W_u^T) (Eq. 5 and the
// summand of Eq. 3) fused with the unembedding product, the exit test of Algorithm 3, and the
// verify-skip gate of Eq. 4.
//
// logit_entropy_kernel: W_u [V][D] bf16 is read exactly once - the kernel is bound by that read.
// Persistent CTAs (one per SM) take 128-row vocabulary tiles round-robin.  Warp 8 streams a tile as
// [128 rows x 64 columns] boxes (16 KiB, 128-byte swizzle) by TMA into a six-stage ring; the
// (up to 16) hidden-state rows sit in shared memory for the whole kernel, loaded once the same way.
// Warps 0-7 each own 16 vocabulary rows of the tile: logits^T = W_tile h^T by mma.sync m16n8k16
// (bf16 in, fp32 accumulate), then an online (max, sum e^(z - max), sum e^(z - max) z) per hidden
// row.  No logit is ever stored.  The per-CTA triples go to a small workspace; a one-block kernel
// merges them: H = max + log Z - S / Z, top-1 probability = 1 / Z.  Waits are bounded.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "kernels.h"

namespace rksc {

namespace {

constexpr int kCgWarps = 8;                       // consumer warps
constexpr int kCgThreads = (kCgWarps + 1) * 32;   // + producer
// Stages of the W ring: six beside 16 hidden rows (112 KiB at D = 3584), ten beside 8 - the kernel
// is bound by HBM latency x bytes in flight, and 96 KiB per SM in flight gives 4.9 TB/s.
template <int NT> struct CgCfg { static constexpr int kStages = NT == 1 ? 10 : 6; };
constexpr int kCgTileRows = 128;                  // vocabulary rows per tile
constexpr int kCgStageBytes = kCgTileRows * 128;  // [128 rows][64 bf16]
constexpr int kCgRows = 16;                       // hidden-state rows per launch

__device__ __forceinline__ uint32_t cg_smem_u32(const void* p) { return static_cast<uint32_t>(__cvta_generic_to_shared(p)); }
__device__ __forceinline__ void cg_mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void cg_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cg_mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
// Bounded wait (2^32 SM cycles), sleeping in hardware between polls.
__device__ __forceinline__ bool cg_mbar_wait(uint32_t bar, uint32_t parity) {
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
            : "r"(bar), "r"(parity), "r"(20000u)
            : "memory");
        if (ok) return true;
        if (clock64() - t0 > (1ll << 32)) return false;
    }
}
__device__ __forceinline__ void cg_tma_2d(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar)
        : "memory");
}
// W_u is read once per call: its lines are the first to leave L2 again.
__device__ __forceinline__ void cg_tma_2d_stream(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar,
                                                 uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
        " [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(tm)), "r"(x), "r"(y), "r"(bar), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void cg_ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
                 : "r"(addr));
}
__device__ __forceinline__ void cg_mma(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

// Running (max, sum e^(z - max), sum e^(z - max) z) of a set of logits, natural units.
struct Stat {
    float m, z, s;
};
__device__ __forceinline__ void stat_add(Stat& a, float v) {
    if (v > a.m) {
        const float f = __expf(a.m - v);   // 0 when a.m = -inf
        a.z = a.z * f + 1.f;
        a.s = a.s * f + v;
        a.m = v;
    } else {
        const float e = __expf(v - a.m);
        a.z += e;
        a.s += e * v;
    }
}
__device__ __forceinline__ Stat stat_merge(const Stat& a, const Stat& b) {
    if (b.z == 0.f) return a;
    if (a.z == 0.f) return b;
    Stat r;
    r.m = fmaxf(a.m, b.m);
    const float fa = __expf(a.m - r.m), fb = __expf(b.m - r.m);
    r.z = a.z * fa + b.z * fb;
    r.s = a.s * fa + b.s * fb;
    return r;
}

template <int NT>
__global__ void __launch_bounds__(kCgThreads, 1)
logit_entropy_kernel(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_h, int D,
                     long long V, float* __restrict__ partial, int32_t* __restrict__ status) {
    extern __shared__ uint8_t cg_smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(cg_smem_raw) + 1023) & ~uintptr_t(1023));
    constexpr int kCgStages = CgCfg<NT>::kStages;
    constexpr int kHChunk = NT * 1024;                     // bytes of one 64-column chunk of the 8 * NT hidden rows
    const int nkc = (D + 63) / 64;                         // 64-column chunks of the hidden dimension
    const uint32_t ring = cg_smem_u32(smem);
    const uint32_t hbase = ring + kCgStages * kCgStageBytes;   // [nkc][8 * NT rows][128 B]
    const uint32_t bars = hbase + nkc * kHChunk;           // full[stages], empty[stages], h
    // per-warp triples of the final merge: over the ring's first stage, which is idle by then
    float (*s_part)[kCgRows][3] = reinterpret_cast<float (*)[kCgRows][3]>(smem);
    __shared__ int s_abort;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if (threadIdx.x == 0) {
        for (int i = 0; i < kCgStages; ++i) {
            cg_mbar_init(bars + 8 * i, 1);
            cg_mbar_init(bars + 8 * (kCgStages + i), kCgWarps);
        }
        cg_mbar_init(bars + 8 * 2 * kCgStages, 1);
        s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    const long long ntiles = (V + kCgTileRows - 1) / kCgTileRows;
    volatile int* abort_flag = &s_abort;
    auto wait_or_abort = [&](uint32_t b, uint32_t parity) {
        if (*abort_flag) return;
        if (!cg_mbar_wait(b, parity)) {
            *abort_flag = 1;
            if (status) atomicExch(status, RKSC_ERR_DEVICE_TIMEOUT);
        }
    };

    if (warp == kCgWarps) {
        // ---------------- producer ----------------
        if (lane == 0) {
            cg_mbar_expect_tx(bars + 8 * 2 * kCgStages, (uint32_t)nkc * (uint32_t)kHChunk);
            for (int kc = 0; kc < nkc; ++kc) cg_tma_2d(hbase + kc * kHChunk, &tm_h, kc * 64, 0, bars + 8 * 2 * kCgStages);
            uint64_t w_policy;
            asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(w_policy));
            uint32_t seq = 0;
            for (long long tile = blockIdx.x; tile < ntiles && !*abort_flag; tile += gridDim.x) {
                for (int kc = 0; kc < nkc && !*abort_flag; ++kc, ++seq) {
                    const uint32_t st = seq % kCgStages;
                    if (seq >= kCgStages) wait_or_abort(bars + 8 * (kCgStages + st), (seq / kCgStages - 1) & 1u);
                    if (*abort_flag) break;
                    cg_mbar_expect_tx(bars + 8 * st, kCgStageBytes);
                    cg_tma_2d_stream(ring + st * kCgStageBytes, &tm_w, kc * 64, (int)(tile * kCgTileRows), bars + 8 * st, w_policy);
                }
            }
        }
    } else {
        // ---------------- consumers ----------------
        const int g4 = lane >> 2, t = lane & 3;
        // ldmatrix lane -> (row, 16-byte chunk) selectors: A operand (W rows), B operand (h rows)
        const int a_row = (((lane >> 3) & 1) << 3) + (lane & 7), a_chunk = lane >> 4;
        const int b_row = ((lane >> 4) << 3) + (lane & 7), b_chunk = (lane >> 3) & 1;
        Stat st[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) st[i] = Stat{-INFINITY, 0.f, 0.f};
        wait_or_abort(bars + 8 * 2 * kCgStages, 0);
        uint32_t seq = 0;
        for (long long tile = blockIdx.x; tile < ntiles && !*abort_flag; tile += gridDim.x) {
            float c0[4] = {0.f, 0.f, 0.f, 0.f}, c1[4] = {0.f, 0.f, 0.f, 0.f};
            for (int kc = 0; kc < nkc; ++kc, ++seq) {
                const uint32_t sg = seq % kCgStages;
                wait_or_abort(bars + 8 * sg, (seq / kCgStages) & 1u);
                if (*abort_flag) break;
                const uint32_t wrow = ring + sg * kCgStageBytes + (16 * warp + a_row) * 128;
                if (NT == 2) {
                    const uint32_t hrow = hbase + kc * kHChunk + b_row * 128;
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        uint32_t a[4], b[4];
                        cg_ldmatrix_x4(wrow + (((ks * 2 + a_chunk) ^ (a_row & 7)) << 4), a);
                        cg_ldmatrix_x4(hrow + (((ks * 2 + b_chunk) ^ (b_row & 7)) << 4), b);
                        cg_mma(c0, a, b[0], b[1]);
                        cg_mma(c1, a, b[2], b[3]);
                    }
                } else {
                    // 8 hidden rows: one ldmatrix.x4 brings the B fragments of two k-steps
                    // (lanes 0-7: k-step 2j low half, 8-15: high half, 16-23 and 24-31: k-step 2j + 1)
                    const uint32_t hrow = hbase + kc * kHChunk + (lane & 7) * 128;
#pragma unroll
                    for (int j = 0; j < 2; ++j) {
                        uint32_t b[4], a0[4], a1[4];
                        cg_ldmatrix_x4(hrow + ((((j * 4) + (lane >> 3)) ^ (lane & 7)) << 4), b);
                        cg_ldmatrix_x4(wrow + ((((2 * j) * 2 + a_chunk) ^ (a_row & 7)) << 4), a0);
                        cg_ldmatrix_x4(wrow + ((((2 * j + 1) * 2 + a_chunk) ^ (a_row & 7)) << 4), a1);
                        cg_mma(c0, a0, b[0], b[1]);
                        cg_mma(c0, a1, b[2], b[3]);
                    }
                }
                __syncwarp();
                if (lane == 0) cg_mbar_arrive(bars + 8 * (kCgStages + sg));
            }
            if (*abort_flag) break;
            // logits of vocabulary rows v0 + g4 and v0 + g4 + 8 for hidden rows 2t, 2t+1, 8+2t, 9+2t
            const long long v0 = tile * kCgTileRows + 16 * warp + g4;
            if (v0 < V) {
                stat_add(st[0], c0[0]);
                stat_add(st[1], c0[1]);
                if (NT == 2) {
                    stat_add(st[2], c1[0]);
                    stat_add(st[3], c1[1]);
                }
            }
            if (v0 + 8 < V) {
                stat_add(st[0], c0[2]);
                stat_add(st[1], c0[3]);
                if (NT == 2) {
                    stat_add(st[2], c1[2]);
                    stat_add(st[3], c1[3]);
                }
            }
        }
        // the eight lanes with the same t hold disjoint vocabulary rows of the same hidden rows
#pragma unroll
        for (int i = 0; i < 4; ++i) {
#pragma unroll
            for (int sh = 4; sh <= 16; sh <<= 1) {
                Stat o;
                o.m = __shfl_xor_sync(0xffffffffu, st[i].m, sh);
                o.z = __shfl_xor_sync(0xffffffffu, st[i].z, sh);
                o.s = __shfl_xor_sync(0xffffffffu, st[i].s, sh);
                st[i] = stat_merge(st[i], o);
            }
        }
        // every stage this warp was given has been consumed; the other warps' stages are not stage 0's
        // memory only if they are done too, so meet before writing over the ring
        asm volatile("bar.sync 1, %0;" ::"n"(kCgWarps * 32) : "memory");
        if (g4 == 0) {
            const int rows[4] = {2 * t, 2 * t + 1, 8 + 2 * t, 9 + 2 * t};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                s_part[warp][rows[i]][0] = st[i].m;
                s_part[warp][rows[i]][1] = st[i].z;
                s_part[warp][rows[i]][2] = st[i].s;
            }
        }
    }
    __syncthreads();
    if (threadIdx.x < kCgRows) {
        Stat a{-INFINITY, 0.f, 0.f};
        for (int w = 0; w < kCgWarps; ++w)
            a = stat_merge(a, Stat{s_part[w][threadIdx.x][0], s_part[w][threadIdx.x][1], s_part[w][threadIdx.x][2]});
        float* dst = partial + ((size_t)blockIdx.x * kCgRows + threadIdx.x) * 3;
        dst[0] = a.m;
        dst[1] = a.z;
        dst[2] = a.s;
    }
}

// One block: thread b merges the CTAs' triples of hidden row b (in CTA order).
__global__ void logit_entropy_finish_kernel(const float* __restrict__ partial, int nparts, int B, float* __restrict__ entropy,
                                            float* __restrict__ top1) {
    const int b = threadIdx.x;
    if (b >= B) return;
    Stat a{-INFINITY, 0.f, 0.f};
    for (int p = 0; p < nparts; ++p) {
        const float* src = partial + ((size_t)p * kCgRows + b) * 3;
        a = stat_merge(a, Stat{src[0], src[1], src[2]});
    }
    // H = -sum p log p = log sum e^z - sum p z = (m + log Z) - S / Z;  max_v p_v = e^(m - m - log Z) = 1 / Z
    if (entropy) entropy[b] = a.z > 0.f ? (a.m + logf(a.z)) - a.s / a.z : __int_as_float(0x7fc00000);
    if (top1) top1[b] = a.z > 0.f ? 1.f / a.z : __int_as_float(0x7fc00000);
}

__global__ void entropy_exit_kernel(const float* __restrict__ H, const float* __restrict__ H_prev, int B, int layer,
                                    int l_min, float theta, float eps, int32_t* __restrict__ flags) {
    const int b = blockIdx.x * blockDim.x + threadIdx.x;
    if (b >= B) return;
    const float h = H[b], hp = H_prev[b];
    flags[b] = (layer >= l_min && h < theta && fabsf(h - hp) < eps) ? 1 : 0;
}

// One block of 256 threads: p[b] = mean over the t steps (summed in step order), then the gate.
__global__ void verify_skip_kernel(const float* __restrict__ top1_steps, int t, int B, float tau_conf, float r_gap,
                                   float* __restrict__ p_out, int32_t* __restrict__ skip) {
    __shared__ float s_top[256], s_second[256];
    float top = -INFINITY, second = -INFINITY;
    for (int b = threadIdx.x; b < B; b += blockDim.x) {
        float acc = 0.f;
        for (int j = 0; j < t; ++j) acc += top1_steps[(size_t)j * B + b];
        const float p = acc / (float)t;
        if (p_out) p_out[b] = p;
        if (p > top) {
            second = top;
            top = p;
        } else if (p > second) {
            second = p;
        }
    }
    s_top[threadIdx.x] = top;
    s_second[threadIdx.x] = second;
    __syncthreads();
    if (threadIdx.x == 0) {
        float T = -INFINITY, S2 = -INFINITY;
        for (int i = 0; i < (int)blockDim.x; ++i) {   // two largest of the union of the threads' pairs
            const float a = s_top[i], c = s_second[i];
            if (a > T) {
                S2 = fmaxf(T, c);
                T = a;
            } else {
                S2 = fmaxf(S2, a);
            }
        }
        if (B == 1) S2 = 0.f;   // no competitor
        *skip = (B >= 1 && T > 0.f && T >= tau_conf && (T - S2) / T >= r_gap) ? 1 : 0;
    }
}

}  // namespace

size_t cgee_smem_bytes(int D, int B) {
    const int nt = B <= 8 ? 1 : 2;
    const int stages = nt == 1 ? CgCfg<1>::kStages : CgCfg<2>::kStages;
    return (size_t)stages * kCgStageBytes + (size_t)((D + 63) / 64) * nt * 1024 + (2 * stages + 1) * 8 + 1024 + 64;
}
int cgee_rows_per_launch() { return kCgRows; }

cudaError_t configure_cgee_kernel(int max_smem) {
    cudaError_t e = cudaFuncSetAttribute(logit_entropy_kernel<1>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
    if (e != cudaSuccess) return e;
    return cudaFuncSetAttribute(logit_entropy_kernel<2>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem);
}

cudaError_t launch_logit_entropy(const CUtensorMap& tm_w, const CUtensorMap& tm_h, int B, int D, long long V, int grid,
                                 float* partial, float* entropy, float* top1, int32_t* status, cudaStream_t stream) {
    if (B <= 8) logit_entropy_kernel<1><<<grid, kCgThreads, cgee_smem_bytes(D, B), stream>>>(tm_w, tm_h, D, V, partial, status);
    else logit_entropy_kernel<2><<<grid, kCgThreads, cgee_smem_bytes(D, B), stream>>>(tm_w, tm_h, D, V, partial, status);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    logit_entropy_finish_kernel<<<1, kCgRows, 0, stream>>>(partial, grid, B, entropy, top1);
    return cudaGetLastError();
}

cudaError_t launch_entropy_exit(const float* H, const float* H_prev, int B, int layer, int l_min, float theta, float eps,
                                int32_t* flags, cudaStream_t stream) {
    if (B <= 0) return cudaSuccess;
    entropy_exit_kernel<<<(B + 127) / 128, 128, 0, stream>>>(H, H_prev, B, layer, l_min, theta, eps, flags);
    return cudaGetLastError();
}

cudaError_t launch_verify_skip(const float* top1_steps, int t, int B, float tau_conf, float r_gap, float* p_out,
                               int32_t* skip, cudaStream_t stream) {
    verify_skip_kernel<<<1, 256, 0, stream>>>(top1_steps, t, B, tau_conf, r_gap, p_out, skip);
    return cudaGetLastError();
}

}  // namespace rksc
