// C ABI entry points: argument checks, plan upload, tensor maps, launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cmath>
#include <cstring>
#include <mutex>
#include <new>

#include "kernels.h"

namespace {

using namespace rksc;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_mu;
thread_local cudaError_t g_last_cuda = cudaSuccess;   // the CUDA error behind the last RKSC_ERR_CUDA of this thread

EncodeTiledFn g_encode = nullptr;
constexpr int kMaxDevices = 64;
int g_dev_state[kMaxDevices];   // 0 unknown, 1 ready (sm_100 family, kernels configured), -1 unsupported, -2 cuda error

// Current device checked once: compute capability 10.x and kernel attributes set.
int32_t ensure_device(int* dev_out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    if (dev_out) *dev_out = dev;
    if (dev < 0 || dev >= kMaxDevices) return RKSC_ERR_UNSUPPORTED;
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_dev_state[dev] == 0) {
        int major = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) {
            cudaGetLastError();
            g_dev_state[dev] = -2;
        } else if (major != 10) {
            g_dev_state[dev] = -1;
        } else if (configure_attention_kernels() != cudaSuccess) {
            cudaGetLastError();
            g_dev_state[dev] = -2;
        } else {
            g_dev_state[dev] = 1;
        }
    }
    if (g_dev_state[dev] == 1) return RKSC_OK;
    return g_dev_state[dev] == -1 ? RKSC_ERR_UNSUPPORTED : RKSC_ERR_CUDA;
}

int32_t get_encode(EncodeTiledFn* fn) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_encode) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) != cudaSuccess ||
            qres != cudaDriverEntryPointSuccess || !p) {
            cudaGetLastError();
            return RKSC_ERR_CUDA;
        }
        g_encode = reinterpret_cast<EncodeTiledFn>(p);
    }
    *fn = g_encode;
    return RKSC_OK;
}

// The pool viewed as a 2-D bf16 tensor [num_pool_blocks * Hkv * 16 rows][head_dim], fetched in
// boxes of 16 rows x 64 columns (128 bytes) with the 128-byte swizzle.
int32_t make_pool_map(const rksc_layout& L, const void* base, CUtensorMap* tm) {
    EncodeTiledFn enc;
    int32_t st = get_encode(&enc);
    if (st != RKSC_OK) return st;
    const cuuint64_t gdim[2] = {(cuuint64_t)L.head_dim, (cuuint64_t)L.num_pool_blocks * L.num_kv_heads * kBlock};
    const cuuint64_t gstride[1] = {(cuuint64_t)L.head_dim * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kBlock};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RKSC_OK : RKSC_ERR_CUDA;
}

// Device arenas (with a pinned staging buffer each) are recycled between plans: creating and
// destroying a plan per decode step then costs no cudaMalloc / cudaFree.
std::vector<PlanArena> g_arena_pool;            // guarded by g_mu
std::vector<rksc_plan*> g_plan_pool;            // destroyed plan objects, kept for their vectors' capacity
cudaStream_t g_upload_stream[kMaxDevices];      // non-blocking: uploads do not wait for the caller's kernels

int32_t acquire_arena(int dev, size_t bytes, PlanArena* out) {
    {
        std::lock_guard<std::mutex> lock(g_mu);
        // the smallest arena that fits and whose last plan has left the GPU: taking one that is still in
        // use would make the caller wait for that plan's kernels (a decode loop that builds step i + 1's
        // plan while step i runs would fall back into step with the GPU); rather a new arena then
        int best = -1;
        for (int i = 0; i < (int)g_arena_pool.size(); ++i) {
            PlanArena& c = g_arena_pool[i];
            if (c.device != dev || c.capacity < bytes) continue;
            if (c.busy) {
                if (cudaEventQuery(c.done) != cudaSuccess) {
                    cudaGetLastError();   // cudaErrorNotReady
                    continue;
                }
                c.busy = false;
            }
            if (best < 0 || c.capacity < g_arena_pool[best].capacity) best = i;
        }
        if (best >= 0) {
            *out = g_arena_pool[best];
            g_arena_pool.erase(g_arena_pool.begin() + best);
        } else {
            *out = PlanArena{};
        }
        if (!g_upload_stream[dev] &&
            cudaStreamCreateWithFlags(&g_upload_stream[dev], cudaStreamNonBlocking) != cudaSuccess) {
            cudaGetLastError();
            return RKSC_ERR_CUDA;
        }
    }
    if (out->dev) {
        // the plan that used this arena last may still have work in flight
        if (out->busy && cudaEventSynchronize(out->done) != cudaSuccess) cudaGetLastError();
        out->busy = false;
        return RKSC_OK;
    }
    size_t cap = 64 << 10;
    while (cap < bytes) cap <<= 1;
    PlanArena a{};
    a.device = dev;
    a.capacity = cap;
    if (cudaMalloc(&a.dev, cap) != cudaSuccess || cudaMallocHost(&a.host, cap) != cudaSuccess ||
        cudaEventCreateWithFlags(&a.done, cudaEventDisableTiming) != cudaSuccess) {
        cudaGetLastError();
        if (a.dev) cudaFree(a.dev);
        if (a.host) cudaFreeHost(a.host);
        return RKSC_ERR_CUDA;
    }
    *out = a;
    return RKSC_OK;
}

void release_arena(PlanArena a, bool used, cudaStream_t last_stream) {
    if (!a.dev) return;
    if (used) {
        a.busy = (cudaEventRecord(a.done, last_stream) == cudaSuccess);
        if (!a.busy) {
            cudaGetLastError();
            cudaStreamSynchronize(last_stream);
        }
    }
    std::lock_guard<std::mutex> lock(g_mu);
    if (g_arena_pool.size() < 16) {
        g_arena_pool.push_back(a);
    } else {
        if (a.busy) cudaEventSynchronize(a.done);
        cudaFree(a.dev);
        cudaFreeHost(a.host);
        cudaEventDestroy(a.done);
    }
}

template <typename T>
size_t bytes_of(const std::vector<T>& v) {
    return (v.size() * sizeof(T) + 255) / 256 * 256;
}

int32_t upload_plan(rksc_plan* p) {
    HostPlan& H = p->host;
    constexpr int kN = 11;
    const size_t sizes[kN] = {bytes_of(H.items),      bytes_of(H.seg_blocks), bytes_of(H.sharers),
                              bytes_of(H.merge_off),  bytes_of(H.merge_rows), bytes_of(H.mass_off),
                              bytes_of(H.br_nblk),    256 /* counters, zeroed */,
                              bytes_of(H.seg_block_off), bytes_of(H.seg_sharer_off), bytes_of(H.score_chunks)};
    size_t total = 0;
    for (size_t s : sizes) total += s;
    if (total == 0) total = 256;
    int32_t st = acquire_arena(p->device, total, &p->arena);
    if (st != RKSC_OK) return st;
    uint8_t* stage = static_cast<uint8_t*>(p->arena.host);
    const void* srcs[kN] = {H.items.data(),      H.seg_blocks.data(), H.sharers.data(),      H.merge_off.data(),
                            H.merge_rows.data(), H.mass_off.data(),   H.br_nblk.data(),      nullptr,
                            H.seg_block_off.data(), H.seg_sharer_off.data(), H.score_chunks.data()};
    const size_t raw[kN] = {H.items.size() * sizeof(WorkItem), H.seg_blocks.size() * 4, H.sharers.size() * sizeof(Sharer),
                            H.merge_off.size() * 4,            H.merge_rows.size() * 4, H.mass_off.size() * 8,
                            H.br_nblk.size() * 4,              0,
                            H.seg_block_off.size() * 4,        H.seg_sharer_off.size() * 4,
                            H.score_chunks.size() * 4};
    size_t offs[kN], off = 0;
    for (int i = 0; i < kN; ++i) {
        offs[i] = off;
        if (raw[i]) std::memcpy(stage + off, srcs[i], raw[i]);
        else std::memset(stage + off, 0, sizes[i]);
        off += sizes[i];
    }
    void* d = p->arena.dev;
    cudaStream_t us = g_upload_stream[p->device];
    if (cudaMemcpyAsync(d, stage, total, cudaMemcpyHostToDevice, us) != cudaSuccess ||
        cudaStreamSynchronize(us) != cudaSuccess) {
        cudaGetLastError();
        release_arena(p->arena, false, nullptr);
        p->arena = PlanArena{};
        return RKSC_ERR_CUDA;
    }
    uint8_t* base = static_cast<uint8_t*>(d);
    p->dev.items = reinterpret_cast<const WorkItem*>(base + offs[0]);
    p->dev.seg_blocks = reinterpret_cast<const int32_t*>(base + offs[1]);
    p->dev.sharers = reinterpret_cast<const Sharer*>(base + offs[2]);
    p->dev.merge_off = reinterpret_cast<const int32_t*>(base + offs[3]);
    p->dev.merge_rows = reinterpret_cast<const int32_t*>(base + offs[4]);
    p->dev.mass_off = reinterpret_cast<const int64_t*>(base + offs[5]);
    p->dev.br_nblk = reinterpret_cast<const int32_t*>(base + offs[6]);
    p->dev.counters = reinterpret_cast<int32_t*>(base + offs[7]);
    p->dev.seg_block_off = reinterpret_cast<const int32_t*>(base + offs[8]);
    p->dev.seg_sharer_off = reinterpret_cast<const int32_t*>(base + offs[9]);
    p->dev.score_chunks = reinterpret_cast<const int32_t*>(base + offs[10]);
    p->on_device = true;
    return RKSC_OK;
}

}  // namespace

extern "C" RKSC_API const char* rksc_strerror(int32_t status) {
    switch (status) {
        case RKSC_OK: return "ok";
        case RKSC_ERR_INVALID_ARG: return "invalid argument";
        case RKSC_ERR_UNSUPPORTED: return "unsupported configuration or device";
        case RKSC_ERR_BAD_TABLE: return "inconsistent block table";
        case RKSC_ERR_WORKSPACE: return "workspace too small or misaligned";
        case RKSC_ERR_CUDA: return "CUDA call failed or no device";
        case RKSC_ERR_DEVICE_TIMEOUT: return "a bounded wait inside a kernel ran out";
        case RKSC_ERR_NOMEM: return "out of host memory";
        default: return "unknown status";
    }
}

extern "C" RKSC_API int32_t rksc_asks_gate(const float* h_branch, const float* h_root, const int32_t* cand_prefix,
                                  int32_t B, int32_t P, int32_t L, int32_t D, float alpha, float tau,
                                  int32_t* branch_to_prefix, float* sigma, void* stream) {
    if (B < 0 || P <= 0 || L <= 0 || D <= 0) return RKSC_ERR_INVALID_ARG;
    if (B == 0) return RKSC_OK;
    if (!h_branch || !h_root || !cand_prefix || !branch_to_prefix) return RKSC_ERR_INVALID_ARG;
    if (!(alpha == alpha) || !(tau == tau)) return RKSC_ERR_INVALID_ARG;
    if ((int64_t)B * 8 >= ((int64_t)1 << 31)) return RKSC_ERR_UNSUPPORTED;
    int32_t st = ensure_device(nullptr);
    if (st != RKSC_OK) return st;
    cudaError_t e = launch_asks_gate(h_branch, h_root, cand_prefix, B, P, L, D, alpha, tau, branch_to_prefix, sigma,
                                     static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    return RKSC_OK;
}

extern "C" RKSC_API const char* rksc_last_cuda_error(void) { return cudaGetErrorString(g_last_cuda); }

extern "C" RKSC_API int32_t rksc_plan_create(const rksc_layout* layout, const rksc_tables* tables, rksc_plan** out) {
    if (!layout || !tables || !out) return RKSC_ERR_INVALID_ARG;
    *out = nullptr;
    rksc_plan* p = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (!g_plan_pool.empty()) {
            p = g_plan_pool.back();
            g_plan_pool.pop_back();
        }
    }
    if (!p) p = new (std::nothrow) rksc_plan();
    if (!p) return RKSC_ERR_NOMEM;
    p->dev = DevicePlan{};
    p->arena = PlanArena{};
    p->used = false;
    p->last_stream = nullptr;
    p->device = -1;
    p->num_sms = 148;
    p->on_device = false;
    int ndev = 0;
    const bool have_dev = (cudaGetDeviceCount(&ndev) == cudaSuccess && ndev > 0);
    if (!have_dev) cudaGetLastError();
    int32_t st = RKSC_OK;
    if (have_dev) {
        st = ensure_device(&p->device);
        if (st == RKSC_OK) {
            int sms = 0;
            if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, p->device) == cudaSuccess && sms > 0)
                p->num_sms = sms;
        }
    }
    if (st == RKSC_OK) {
        try {
            st = build_host_plan(*layout, *tables, p->num_sms, &p->host);
        } catch (const std::bad_alloc&) {
            st = RKSC_ERR_NOMEM;
        }
    }
    if (st == RKSC_OK && have_dev) st = upload_plan(p);
    if (st != RKSC_OK) {
        delete p;
        return st;
    }
    *out = p;
    return RKSC_OK;
}

extern "C" RKSC_API int32_t rksc_plan_create_from_gate(
    const rksc_layout* layout, int32_t B, int32_t P, const int32_t* branch_to_prefix, const int32_t* shared_off,
    const int32_t* shared_pages, const int32_t* shared_ntok, const int32_t* priv_off, const int32_t* priv_pages,
    const int32_t* priv_ntok, const int32_t* sfx_off, const int32_t* sfx_pages, const int32_t* sfx_ntok,
    rksc_plan** out) {
    if (!out) return RKSC_ERR_INVALID_ARG;
    *out = nullptr;
    rksc_tables t;
    int32_t st = rksc_tables_from_gate(B, P, branch_to_prefix, shared_off, shared_pages, shared_ntok, priv_off,
                                       priv_pages, priv_ntok, sfx_off, sfx_pages, sfx_ntok, &t);
    if (st != RKSC_OK) return st;
    st = rksc_plan_create(layout, &t, out);
    rksc_tables_free(&t);
    return st;
}

extern "C" RKSC_API int32_t rksc_plan_query(const rksc_plan* plan, rksc_plan_info* info) {
    if (!plan || !info) return RKSC_ERR_INVALID_ARG;
    const HostPlan& H = plan->host;
    info->workspace_bytes = H.workspace_bytes;
    info->mass_elems = H.mass_elems;
    info->mass_off = H.mass_off.data();
    info->num_work_items = H.num_work_items;
    info->num_partial_rows = H.num_partial_rows;
    info->unique_kv_tokens = H.unique_kv_tokens;
    info->duplicated_kv_tokens = H.duplicated_kv_tokens;
    info->on_device = plan->on_device ? 1 : 0;
    info->num_pages_listed = (int64_t)H.seg_blocks.size();
    info->num_kernel_launches = H.B == 0 ? 0 : (H.num_tc_items > 0 ? 1 : 0) +
                                                   (H.num_work_items > H.num_tc_items ? 1 : 0) + 1;
    return RKSC_OK;
}

extern "C" RKSC_API int32_t rksc_plan_get_item(const rksc_plan* plan, int32_t i, int32_t* out10) {
    if (!plan || !out10) return RKSC_ERR_INVALID_ARG;
    const HostPlan& H = plan->host;
    if (i < 0 || i >= H.num_work_items) return RKSC_ERR_INVALID_ARG;
    const WorkItem it = work_item_of(H.items.data(), i, H.layout.num_kv_heads, H.G);
    out10[0] = it.seg;
    out10[1] = it.kv_head;
    out10[2] = it.seg_page_begin;
    out10[3] = it.num_pages;
    out10[4] = it.num_tokens;
    out10[5] = it.sharer_begin - H.seg_sharer_off[it.seg];
    out10[6] = it.num_sharers;
    out10[7] = it.part_row_base;
    out10[8] = it.klass;
    out10[9] = 0;
    return RKSC_OK;
}

extern "C" RKSC_API void rksc_plan_destroy(rksc_plan* plan) {
    if (!plan) return;
    if (plan->arena.dev) {
        int cur = -1;
        const bool sw = (cudaGetDevice(&cur) == cudaSuccess && cur != plan->device && plan->device >= 0);
        if (sw) cudaSetDevice(plan->device);
        release_arena(plan->arena, plan->used, static_cast<cudaStream_t>(plan->last_stream));
        if (sw) cudaSetDevice(cur);
    }
    {
        std::lock_guard<std::mutex> lock(g_mu);
        if (g_plan_pool.size() < 8) {
            g_plan_pool.push_back(plan);
            return;
        }
    }
    delete plan;
}

extern "C" RKSC_API int32_t rksc_branch_decode_attention(const rksc_plan* plan, const void* q, const void* k_pool,
                                                const void* v_pool, float* out, float* block_mass, void* workspace,
                                                size_t workspace_bytes, int32_t* device_status, void* stream) {
    return rksc_branch_decode_attention_phases(plan, q, k_pool, v_pool, out, block_mass, workspace, workspace_bytes,
                                               device_status, stream, RKSC_PHASE_SEGMENTS | RKSC_PHASE_MERGE);
}

extern "C" RKSC_API int32_t rksc_branch_decode_attention_phases(const rksc_plan* plan, const void* q,
                                                const void* k_pool, const void* v_pool, float* out,
                                                float* block_mass, void* workspace, size_t workspace_bytes,
                                                int32_t* device_status, void* stream, int32_t phases) {
    if (!plan) return RKSC_ERR_INVALID_ARG;
    if ((phases & ~(RKSC_PHASE_SEGMENTS | RKSC_PHASE_MERGE | RKSC_PHASE_MERGE_LATE)) ||
        (phases & (RKSC_PHASE_SEGMENTS | RKSC_PHASE_MERGE)) == 0)
        return RKSC_ERR_INVALID_ARG;
    const HostPlan& H = plan->host;
    if (H.B == 0) return RKSC_OK;
    if (!q || !k_pool || !v_pool || !out) return RKSC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(q) & 15) || (reinterpret_cast<uintptr_t>(k_pool) & 15) ||
        (reinterpret_cast<uintptr_t>(v_pool) & 15) || (reinterpret_cast<uintptr_t>(out) & 15))
        return RKSC_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < H.workspace_bytes || (reinterpret_cast<uintptr_t>(workspace) & 255))
        return RKSC_ERR_WORKSPACE;
    if (!plan->on_device) return RKSC_ERR_CUDA;
    int dev = -1;
    int32_t st = ensure_device(&dev);
    if (st != RKSC_OK) return st;
    if (dev != plan->device) return RKSC_ERR_INVALID_ARG;

    CUtensorMap tm_k, tm_v;
    st = make_pool_map(H.layout, k_pool, &tm_k);
    if (st != RKSC_OK) return st;
    st = make_pool_map(H.layout, v_pool, &tm_v);
    if (st != RKSC_OK) return st;

    AttnArgs a{};
    a.plan = plan->dev;
    a.q = q;
    a.part_o = static_cast<float*>(workspace);
    a.part_lse = reinterpret_cast<float*>(static_cast<uint8_t*>(workspace) + H.ws_lse_offset);
    a.block_mass = block_mass;
    a.out = out;
    a.status = device_status;
    a.counters = plan->dev.counters;
    a.num_items = H.num_work_items;
    a.num_tc_items = H.num_tc_items;
    a.grid_warp = H.grid_warp;
    a.grid_tc = H.grid_tc;
    a.B = H.B;
    a.Hq = H.layout.num_q_heads;
    a.Hkv = H.layout.num_kv_heads;
    a.G = H.G;
    a.head_dim = H.layout.head_dim;
    const float scale = H.layout.sm_scale > 0.f ? H.layout.sm_scale : 1.0f / std::sqrt((float)H.layout.head_dim);
    a.scale_log2 = scale * 1.4426950408889634f;

    cudaStream_t s = static_cast<cudaStream_t>(stream);
    plan->used = true;
    plan->last_stream = stream;
    cudaError_t e = cudaSuccess;
    if (phases & RKSC_PHASE_SEGMENTS) {
        e = launch_seg_attn_tc(tm_k, tm_v, a, s);
        if (e == cudaSuccess) e = launch_seg_attn_warp(tm_k, tm_v, a, s, /*after_tc=*/a.grid_tc > 0);
    }
    if (e == cudaSuccess && (phases & RKSC_PHASE_MERGE)) e = launch_merge(a, s, !(phases & RKSC_PHASE_MERGE_LATE));
    if (e != cudaSuccess) {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    return RKSC_OK;
}

// ---------------------------------------------------------------------------------------------
// The whole path for host-resident inputs (KV pool resident on the device)
// ---------------------------------------------------------------------------------------------

namespace {

// The per-step device buffers come from a memory pool of the library's own, one per device, that
// keeps what is freed: the device's default pool hands freed memory back to the system at every
// synchronisation (release threshold 0), and mapping a hundred megabytes anew each step costs
// milliseconds.  The pool holds about one step's buffers between calls.
cudaMemPool_t g_step_pool[kMaxDevices];
bool g_step_pool_ready[kMaxDevices];

cudaError_t step_pool(int dev, cudaMemPool_t* pool) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_step_pool_ready[dev]) {
        cudaMemPoolProps props = {};
        props.allocType = cudaMemAllocationTypePinned;
        props.handleTypes = cudaMemHandleTypeNone;
        props.location.type = cudaMemLocationTypeDevice;
        props.location.id = dev;
        cudaError_t e = cudaMemPoolCreate(&g_step_pool[dev], &props);
        if (e != cudaSuccess) return e;
        uint64_t keep = UINT64_MAX;
        e = cudaMemPoolSetAttribute(g_step_pool[dev], cudaMemPoolAttrReleaseThreshold, &keep);
        if (e != cudaSuccess) return e;
        g_step_pool_ready[dev] = true;
    }
    *pool = g_step_pool[dev];
    return cudaSuccess;
}

struct AsyncBuf {   // stream-ordered device buffer, released on scope exit
    void* p = nullptr;
    cudaStream_t s = nullptr;
    cudaMemPool_t pool = nullptr;
    cudaError_t alloc(size_t bytes, cudaStream_t stream) {
        s = stream;
        return cudaMallocFromPoolAsync(&p, bytes ? bytes : 16, pool, stream);
    }
    ~AsyncBuf() {
        if (p) cudaFreeAsync(p, s);
    }
};

}  // namespace

extern "C" RKSC_API int32_t rksc_decode_step_host(
    const rksc_layout* layout, const float* h_branch, const float* h_root, const int32_t* cand_prefix, int32_t B,
    int32_t P, int32_t L, int32_t D, float alpha, float tau, const int32_t* shared_off, const int32_t* shared_pages,
    const int32_t* shared_ntok, const int32_t* priv_off, const int32_t* priv_pages, const int32_t* priv_ntok,
    const int32_t* sfx_off, const int32_t* sfx_pages, const int32_t* sfx_ntok, const void* q, const void* k_pool,
    const void* v_pool, int32_t* branch_to_prefix, float* sigma, float* out, float* block_mass,
    int64_t block_mass_capacity, int64_t* mass_off, void* stream) {
    if (!layout || !h_branch || !h_root || !cand_prefix || !q || !k_pool || !v_pool || !branch_to_prefix || !out)
        return RKSC_ERR_INVALID_ARG;
    if (B <= 0 || P <= 0 || L <= 0 || D <= 0) return RKSC_ERR_INVALID_ARG;
    int dev = -1;
    int32_t st = ensure_device(&dev);
    if (st != RKSC_OK) return st;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaMemPool_t pool = nullptr;
    if (step_pool(dev, &pool) != cudaSuccess) {
        g_last_cuda = cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    const size_t nb = (size_t)B * L * D * sizeof(float), nr = (size_t)P * L * D * sizeof(float);
    const size_t nq = (size_t)B * layout->num_q_heads * layout->head_dim * 2;
    const size_t nout = (size_t)B * layout->num_q_heads * layout->head_dim * sizeof(float);
    AsyncBuf d_hb, d_hr, d_cand, d_map, d_sigma, d_q, d_out, d_mass, d_ws, d_status;
    for (AsyncBuf* b : {&d_hb, &d_hr, &d_cand, &d_map, &d_sigma, &d_q, &d_out, &d_mass, &d_ws, &d_status}) b->pool = pool;
    cudaError_t e = cudaSuccess;
    auto ok = [&](cudaError_t r) {
        if (e == cudaSuccess && r != cudaSuccess) e = r;
        return e == cudaSuccess;
    };
    auto fail = [&]() {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    };
    // gate: inputs to the device, kernel, map (and sigma) back
    if (!ok(d_hb.alloc(nb, s)) || !ok(d_hr.alloc(nr, s)) || !ok(d_cand.alloc((size_t)B * 4, s)) ||
        !ok(d_map.alloc((size_t)B * 4, s)) || !ok(d_sigma.alloc((size_t)B * 4, s)) || !ok(d_q.alloc(nq, s)) ||
        !ok(d_out.alloc(nout, s)) || !ok(d_status.alloc(16, s)))
        return fail();
    ok(cudaMemcpyAsync(d_hb.p, h_branch, nb, cudaMemcpyHostToDevice, s));
    ok(cudaMemcpyAsync(d_hr.p, h_root, nr, cudaMemcpyHostToDevice, s));
    ok(cudaMemcpyAsync(d_cand.p, cand_prefix, (size_t)B * 4, cudaMemcpyHostToDevice, s));
    ok(cudaMemcpyAsync(d_q.p, q, nq, cudaMemcpyHostToDevice, s));
    ok(cudaMemsetAsync(d_status.p, 0, 16, s));
    if (e != cudaSuccess) return fail();
    st = rksc_asks_gate((const float*)d_hb.p, (const float*)d_hr.p, (const int32_t*)d_cand.p, B, P, L, D, alpha, tau,
                        (int32_t*)d_map.p, (float*)d_sigma.p, stream);
    if (st != RKSC_OK) return st;
    ok(cudaMemcpyAsync(branch_to_prefix, d_map.p, (size_t)B * 4, cudaMemcpyDeviceToHost, s));
    if (sigma) ok(cudaMemcpyAsync(sigma, d_sigma.p, (size_t)B * 4, cudaMemcpyDeviceToHost, s));
    ok(cudaStreamSynchronize(s));   // the tables are built on the host from the map
    if (e != cudaSuccess) return fail();

    rksc_tables tables;
    st = rksc_tables_from_gate(B, P, branch_to_prefix, shared_off, shared_pages, shared_ntok, priv_off, priv_pages,
                               priv_ntok, sfx_off, sfx_pages, sfx_ntok, &tables);
    if (st != RKSC_OK) return st;
    rksc_plan* plan = nullptr;
    st = rksc_plan_create(layout, &tables, &plan);
    rksc_tables_free(&tables);
    if (st != RKSC_OK) return st;
    const HostPlan& H = plan->host;
    if (mass_off) std::memcpy(mass_off, H.mass_off.data(), (size_t)(B + 1) * sizeof(int64_t));
    if (block_mass && block_mass_capacity < H.mass_elems) {
        rksc_plan_destroy(plan);
        return RKSC_ERR_INVALID_ARG;
    }
    if (!ok(d_ws.alloc(H.workspace_bytes, s)) || (block_mass && !ok(d_mass.alloc((size_t)H.mass_elems * 4, s)))) {
        rksc_plan_destroy(plan);
        return fail();
    }
    st = rksc_branch_decode_attention(plan, d_q.p, k_pool, v_pool, (float*)d_out.p, block_mass ? (float*)d_mass.p : nullptr,
                                      d_ws.p, H.workspace_bytes, (int32_t*)d_status.p, stream);
    int32_t dev_status = 0;
    if (st == RKSC_OK) {
        ok(cudaMemcpyAsync(out, d_out.p, nout, cudaMemcpyDeviceToHost, s));
        if (block_mass) ok(cudaMemcpyAsync(block_mass, d_mass.p, (size_t)H.mass_elems * 4, cudaMemcpyDeviceToHost, s));
        ok(cudaMemcpyAsync(&dev_status, d_status.p, 4, cudaMemcpyDeviceToHost, s));
    }
    ok(cudaStreamSynchronize(s));   // also ends the plan's use before it is destroyed
    rksc_plan_destroy(plan);
    if (st != RKSC_OK) return st;
    if (e != cudaSuccess) return fail();
    return dev_status;
}

// ---------------------------------------------------------------------------------------------
// Attention without any allocation by the caller: the partial-result scratch lives in the library
// ---------------------------------------------------------------------------------------------

namespace {

// The scratch the segment kernels write their partial results to and the merge kernel reads them
// from.  It is part of the loaded module: every GPU that loads this library keeps these bytes
// until the process exits.
static __device__ __align__(256) unsigned char g_static_workspace[RKSC_STATIC_WORKSPACE_BYTES];

// In host code the array's name is only a handle for the runtime, not a device address; the address
// the kernels need is asked for once per device and kept here.
void* g_static_workspace_ptr[kMaxDevices];

int32_t static_workspace(int dev, void** out) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_static_workspace_ptr[dev]) {
        void* p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress(&p, g_static_workspace);   // for the current device
        if (e != cudaSuccess || !p) {
            g_last_cuda = e;
            cudaGetLastError();
            return RKSC_ERR_CUDA;
        }
        g_static_workspace_ptr[dev] = p;
    }
    *out = g_static_workspace_ptr[dev];
    return RKSC_OK;
}

}  // namespace

extern "C" RKSC_API int32_t rksc_branch_decode_attention_static(const rksc_plan* plan, const void* q,
                                                               const void* k_pool, const void* v_pool, float* out,
                                                               float* block_mass, int32_t* device_status,
                                                               void* stream) {
    if (!plan) return RKSC_ERR_INVALID_ARG;
    if (plan->host.workspace_bytes > (size_t)RKSC_STATIC_WORKSPACE_BYTES) return RKSC_ERR_WORKSPACE;
    if (plan->host.B == 0) return RKSC_OK;
    int dev = -1;
    int32_t st = ensure_device(&dev);
    if (st != RKSC_OK) return st;
    void* ws = nullptr;
    st = static_workspace(dev, &ws);
    if (st != RKSC_OK) return st;
    return rksc_branch_decode_attention(plan, q, k_pool, v_pool, out, block_mass, ws,
                                        (size_t)RKSC_STATIC_WORKSPACE_BYTES, device_status, stream);
}

// ---- RSBCM eviction (Section 2.4, Algorithm 4) ----

extern "C" RKSC_API int32_t rksc_rsbcm_page_scores(const rksc_plan* plan, const float* block_mass, double* score,
                                                   void* stream) {
    if (!plan) return RKSC_ERR_INVALID_ARG;
    const HostPlan& H = plan->host;
    const int num_chunks = (int)(H.score_chunks.size() / 2);
    if (num_chunks == 0) return RKSC_OK;
    if (!block_mass || !score || !plan->on_device) return RKSC_ERR_INVALID_ARG;
    int32_t st = ensure_device(nullptr);
    if (st != RKSC_OK) return st;
    cudaError_t e = launch_page_scores(reinterpret_cast<const int2*>(plan->dev.score_chunks), num_chunks,
                                       plan->dev.seg_block_off, plan->dev.seg_sharer_off, plan->dev.sharers, block_mass,
                                       score, H.layout.num_q_heads, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    return RKSC_OK;
}

extern "C" RKSC_API size_t rksc_rsbcm_workspace_bytes(int64_t n) {
    if (n < 0) n = 0;
    const size_t b = ((size_t)n * 8 + 255) / 256 * 256;
    return b ? b : 256;
}

extern "C" RKSC_API int32_t rksc_rsbcm_evict(const double* score, const int32_t* depth, int64_t n, int64_t capacity,
                                             uint8_t* evicted, int32_t* num_evicted, void* workspace,
                                             size_t workspace_bytes, void* stream) {
    if (n < 0 || n >= ((int64_t)1 << 31)) return RKSC_ERR_INVALID_ARG;
    if (n > 0 && (!score || !depth || !evicted)) return RKSC_ERR_INVALID_ARG;
    if (!workspace || workspace_bytes < rksc_rsbcm_workspace_bytes(n) ||
        (reinterpret_cast<uintptr_t>(workspace) & 255) != 0)
        return RKSC_ERR_WORKSPACE;
    if (n == 0 && !num_evicted) return RKSC_OK;
    int32_t st = ensure_device(nullptr);
    if (st != RKSC_OK) return st;
    if (capacity < 0) capacity = 0;
    const uint32_t k = capacity >= n ? 0u : (uint32_t)(n - capacity);
    cudaError_t e = launch_rsbcm_select(score, depth, (int32_t)n, k, static_cast<uint64_t*>(workspace), evicted,
                                        num_evicted, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    return RKSC_OK;
}

// ---- CGEE numerics (Section 2.3: Eq. 3-5, Algorithm 3) ----

namespace {
// A row-major bf16 matrix [rows][cols] fetched in boxes of box_rows x 64 columns, 128-byte swizzle.
int32_t make_matrix_map(const void* base, int64_t rows, int cols, int box_rows, CUtensorMap* tm) {
    EncodeTiledFn enc;
    int32_t st = get_encode(&enc);
    if (st != RKSC_OK) return st;
    const cuuint64_t gdim[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)cols * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)box_rows};
    const cuuint32_t estr[2] = {1, 1};
    CUresult r = enc(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), gdim, gstride, box, estr,
                     CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                     CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? RKSC_OK : RKSC_ERR_CUDA;
}
constexpr int kCgeeMaxParts = 1024;   // CTAs whose partial results the workspace holds
}  // namespace

extern "C" RKSC_API size_t rksc_cgee_workspace_bytes(void) { return (size_t)kCgeeMaxParts * 16 * 3 * sizeof(float); }

extern "C" RKSC_API int32_t rksc_cgee_logit_entropy(const void* h, const void* w_u, int32_t B, int32_t D, int64_t V,
                                                    float* entropy, float* top1_prob, void* workspace,
                                                    size_t workspace_bytes, int32_t* device_status, void* stream) {
    if (B < 0 || D <= 0 || V <= 0) return RKSC_ERR_INVALID_ARG;
    if (B == 0) return RKSC_OK;
    if (!h || !w_u || (!entropy && !top1_prob)) return RKSC_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(h) & 15) || (reinterpret_cast<uintptr_t>(w_u) & 15)) return RKSC_ERR_INVALID_ARG;
    if (D % 8 != 0 || V >= ((int64_t)1 << 31)) return RKSC_ERR_UNSUPPORTED;   // TMA: row pitch a multiple of 16 bytes
    if (!workspace || workspace_bytes < rksc_cgee_workspace_bytes() || (reinterpret_cast<uintptr_t>(workspace) & 15))
        return RKSC_ERR_WORKSPACE;
    int dev = -1;
    int32_t st = ensure_device(&dev);
    if (st != RKSC_OK) return st;
    const size_t smem = cgee_smem_bytes(D, 16);
    if (smem > 227 * 1024 - 256) return RKSC_ERR_UNSUPPORTED;   // the hidden rows must fit in shared memory (D <= 4096)
    static bool configured[kMaxDevices] = {};
    static int sms[kMaxDevices] = {};
    if (!configured[dev]) {
        if (configure_cgee_kernel(227 * 1024 - 256) != cudaSuccess ||
            cudaDeviceGetAttribute(&sms[dev], cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) {
            g_last_cuda = cudaGetLastError();
            return RKSC_ERR_CUDA;
        }
        configured[dev] = true;
    }
    const int64_t ntiles = (V + 127) / 128;
    const int grid = (int)std::min<int64_t>(std::min<int64_t>(ntiles, std::max(1, sms[dev])), kCgeeMaxParts);
    CUtensorMap tm_w;
    st = make_matrix_map(w_u, V, D, 128, &tm_w);
    if (st != RKSC_OK) return st;
    const int rows_per = cgee_rows_per_launch();
    // more rows than one launch takes: row blocks one after another (W_u is read once per block)
    for (int b0 = 0; b0 < B; b0 += rows_per) {
        const int nb = std::min(rows_per, B - b0);
        CUtensorMap tm_h;
        st = make_matrix_map(static_cast<const uint8_t*>(h) + (size_t)b0 * D * 2, nb, D, nb <= 8 ? 8 : rows_per, &tm_h);
        if (st != RKSC_OK) return st;
        cudaError_t e = launch_logit_entropy(tm_w, tm_h, nb, D, V, grid, static_cast<float*>(workspace),
                                             entropy ? entropy + b0 : nullptr, top1_prob ? top1_prob + b0 : nullptr,
                                             device_status, static_cast<cudaStream_t>(stream));
        if (e != cudaSuccess) {
            g_last_cuda = e;
            cudaGetLastError();
            return RKSC_ERR_CUDA;
        }
    }
    return RKSC_OK;
}

extern "C" RKSC_API int32_t rksc_cgee_entropy_exit(const float* entropy, const float* entropy_prev, int32_t B, int32_t layer,
                                                   int32_t l_min, float theta, float eps, int32_t* exit_flags,
                                                   void* stream) {
    if (B < 0) return RKSC_ERR_INVALID_ARG;
    if (B == 0) return RKSC_OK;
    if (!entropy || !entropy_prev || !exit_flags) return RKSC_ERR_INVALID_ARG;
    int32_t st = ensure_device(nullptr);
    if (st != RKSC_OK) return st;
    cudaError_t e = launch_entropy_exit(entropy, entropy_prev, B, layer, l_min, theta, eps, exit_flags,
                                        static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    return RKSC_OK;
}

extern "C" RKSC_API int32_t rksc_cgee_verify_skip(const float* top1_per_step, int32_t t, int32_t B, float tau_conf,
                                                  float r_gap, float* confidence, int32_t* skip, void* stream) {
    if (t < 1 || B < 0 || !skip) return RKSC_ERR_INVALID_ARG;
    if (B > 0 && !top1_per_step) return RKSC_ERR_INVALID_ARG;
    int32_t st = ensure_device(nullptr);
    if (st != RKSC_OK) return st;
    cudaError_t e = launch_verify_skip(top1_per_step, t, B, tau_conf, r_gap, confidence, skip,
                                       static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    return RKSC_OK;
}

// ---- token-by-token decode on the paged cache (Appendix "Stepwise Batched Decode", step 2) ----

extern "C" RKSC_API int32_t rksc_kv_append(const rksc_layout* layout, void* k_pool, void* v_pool, const void* k_new,
                                           const void* v_new, int32_t B, const int32_t* page, const int32_t* slot,
                                           void* stream) {
    if (!layout || B < 0) return RKSC_ERR_INVALID_ARG;
    if (B == 0) return RKSC_OK;
    if (!k_pool || !v_pool || !k_new || !v_new || !page || !slot) return RKSC_ERR_INVALID_ARG;
    if (layout->num_kv_heads <= 0 || layout->head_dim <= 0 || layout->num_pool_blocks <= 0) return RKSC_ERR_INVALID_ARG;
    if (layout->block_size != kBlock) return RKSC_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(k_pool) & 15) || (reinterpret_cast<uintptr_t>(v_pool) & 15) ||
        (reinterpret_cast<uintptr_t>(k_new) & 15) || (reinterpret_cast<uintptr_t>(v_new) & 15))
        return RKSC_ERR_INVALID_ARG;
    int32_t st = ensure_device(nullptr);
    if (st != RKSC_OK) return st;
    cudaError_t e = launch_kv_append(k_pool, v_pool, k_new, v_new, page, slot, B, layout->num_kv_heads, layout->head_dim,
                                     layout->num_pool_blocks, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    return RKSC_OK;
}

// ---------------------------------------------------------------------------------------------
// Self-test of the bounded wait
// ---------------------------------------------------------------------------------------------

extern "C" RKSC_API int32_t rksc_debug_wait_timeout(int64_t limit_cycles, int32_t* device_status, void* stream) {
    if (limit_cycles < 1 || limit_cycles > ((int64_t)1 << 31) || !device_status) return RKSC_ERR_INVALID_ARG;
    int32_t st = ensure_device(nullptr);
    if (st != RKSC_OK) return st;
    const cudaError_t e = launch_wait_timeout((long long)limit_cycles, device_status, static_cast<cudaStream_t>(stream));
    if (e != cudaSuccess) {
        g_last_cuda = e;
        cudaGetLastError();
        return RKSC_ERR_CUDA;
    }
    return RKSC_OK;
}
