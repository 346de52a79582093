// Step pipeline: whole steps of the path kept several deep in flight by the library's own host
// threads (declared in rksc.h).  Everything here goes through the library's public entry points:
// the gate kernel, rksc_plan_create_from_gate, the attention call.
//
// A step occupies a slot (ticket % depth).  The submitting thread enqueues the gate and the copy of
// its map on the gate stream; a worker thread waits for the copy, builds the plan and enqueues the
// attention on the attention stream, workers taking turns in ticket order.
#include <cuda_runtime_api.h>

#include <condition_variable>
#include <cstring>
#include <deque>
#include <initializer_list>
#include <mutex>
#include <new>
#include <thread>
#include <vector>

#include "rksc.h"

namespace {

struct Slot {
    // per-step arguments
    const float* h_branch = nullptr;
    const float* h_root = nullptr;
    const int32_t* cand = nullptr;
    const void* q = nullptr;
    const void* k_pool = nullptr;
    const void* v_pool = nullptr;
    float* out = nullptr;
    float* block_mass = nullptr;
    // owned
    int32_t* map_dev = nullptr;
    float* sigma_dev = nullptr;
    int32_t* status_dev = nullptr;
    int32_t* map_host = nullptr;       // pinned: [B] map, then [B] sigma (as float), then the status word
    void* workspace = nullptr;
    size_t workspace_cap = 0;
    cudaEvent_t ev_map = nullptr;      // gate + map copy done
    cudaEvent_t ev_att = nullptr;      // attention enqueued on the attention stream is done
    cudaEvent_t ev_done = nullptr;     // attention + status copy done
    cudaEvent_t ev_seg0 = nullptr, ev_seg1 = nullptr;   // timing pipelines
    rksc_plan* plan = nullptr;
    int64_t ticket = -1;
    int32_t status = RKSC_OK;          // host-side status of the step's stages
    bool attention_enqueued = false;
    bool timed = false;                // this step's segment kernels have events around them
    bool worker_done = true;           // the slot's worker has finished with it
    bool waited = true;                // rksc_pipeline_wait has returned for its ticket
};

}  // namespace

struct rksc_pipeline {
    rksc_layout layout{};
    int32_t B = 0, P = 0, L = 0, D = 0;
    float alpha = 0.f, tau = 0.f;
    std::vector<int32_t> lists[9];
    int depth = 0;
    int64_t mass_capacity = 0;
    int timing = 0;                    // 0: no events; n > 0: every n-th step (ticket % n == 0) is timed
    int device = -1;
    cudaStream_t gate_stream = nullptr, att_stream = nullptr;
    cudaStream_t copy_stream = nullptr;   // status words back to the host, off the attention stream
    cudaEvent_t ev_inputs = nullptr;
    std::vector<Slot> slots;
    int64_t next_ticket = 0;           // submitting thread only
    int64_t next_wait = 0;             // waiting thread only

    std::mutex mu;
    std::condition_variable cv_jobs, cv_turn, cv_done;
    std::deque<int64_t> jobs;          // tickets whose gate is enqueued
    int64_t next_attention = 0;        // ticket whose attention is enqueued next
    bool stop = false;
    std::vector<std::thread> workers;
};

namespace {

void worker_main(rksc_pipeline* p) {
    cudaSetDevice(p->device);
    for (;;) {
        int64_t t;
        {
            std::unique_lock<std::mutex> lock(p->mu);
            p->cv_jobs.wait(lock, [&] { return p->stop || !p->jobs.empty(); });
            if (p->jobs.empty()) return;   // stop requested and nothing left
            t = p->jobs.front();
            p->jobs.pop_front();
        }
        Slot& s = p->slots[t % p->depth];
        int32_t st = s.status;
        rksc_plan* plan = nullptr;
        rksc_plan_info info{};
        if (st == RKSC_OK && cudaEventSynchronize(s.ev_map) != cudaSuccess) {
            cudaGetLastError();
            st = RKSC_ERR_CUDA;
        }
        if (st == RKSC_OK)
            st = rksc_plan_create_from_gate(&p->layout, p->B, p->P, s.map_host, p->lists[0].data(), p->lists[1].data(),
                                            p->lists[2].data(), p->lists[3].data(), p->lists[4].data(),
                                            p->lists[5].data(), p->lists[6].data(), p->lists[7].data(),
                                            p->lists[8].data(), &plan);
        if (st == RKSC_OK) st = rksc_plan_query(plan, &info);
        if (st == RKSC_OK && s.block_mass != nullptr && info.mass_elems > p->mass_capacity) st = RKSC_ERR_WORKSPACE;
        if (st == RKSC_OK && info.workspace_bytes > s.workspace_cap) {
            // steps differ in their maps, so a later step may need more room than any before it
            if (s.workspace) {
                cudaStreamSynchronize(p->att_stream);
                cudaFree(s.workspace);
                s.workspace = nullptr;
                s.workspace_cap = 0;
            }
            const size_t want = info.workspace_bytes + info.workspace_bytes / 4;
            if (cudaMalloc(&s.workspace, want) != cudaSuccess) {
                cudaGetLastError();
                st = RKSC_ERR_CUDA;
            } else {
                s.workspace_cap = want;
            }
        }
        // attention launches go out in ticket order
        {
            std::unique_lock<std::mutex> lock(p->mu);
            p->cv_turn.wait(lock, [&] { return p->next_attention == t; });
        }
        if (st == RKSC_OK) {
            cudaStream_t as = p->att_stream;
            s.timed = p->timing > 0 && t % p->timing == 0;
            if (s.timed) {
                cudaEventRecord(s.ev_seg0, as);
                st = rksc_branch_decode_attention_phases(plan, s.q, s.k_pool, s.v_pool, s.out, s.block_mass, s.workspace,
                                                         s.workspace_cap, s.status_dev, as, RKSC_PHASE_SEGMENTS);
                cudaEventRecord(s.ev_seg1, as);
                if (st == RKSC_OK)
                    st = rksc_branch_decode_attention_phases(plan, s.q, s.k_pool, s.v_pool, s.out, s.block_mass,
                                                             s.workspace, s.workspace_cap, s.status_dev, as,
                                                             RKSC_PHASE_MERGE | RKSC_PHASE_MERGE_LATE);
            } else {
                // the merge as an ordinary successor: the gate kernels of later steps use the SMs the segment
                // kernel frees while it drains, instead of merge blocks that would only wait there
                st = rksc_branch_decode_attention_phases(plan, s.q, s.k_pool, s.v_pool, s.out, s.block_mass, s.workspace,
                                                         s.workspace_cap, s.status_dev, as,
                                                         RKSC_PHASE_SEGMENTS | RKSC_PHASE_MERGE | RKSC_PHASE_MERGE_LATE);
            }
            s.attention_enqueued = (st == RKSC_OK);
            // The status word goes back on a stream of its own, behind an event: a copy between two steps'
            // kernels on the attention stream would put a copy-engine round trip between them.
            cudaStream_t cs = p->copy_stream;
            if (cudaEventRecord(s.ev_att, as) != cudaSuccess || cudaStreamWaitEvent(cs, s.ev_att, 0) != cudaSuccess ||
                cudaMemcpyAsync(s.map_host + 2 * (size_t)p->B, s.status_dev, sizeof(int32_t), cudaMemcpyDeviceToHost, cs) !=
                    cudaSuccess ||
                cudaEventRecord(s.ev_done, cs) != cudaSuccess) {
                cudaGetLastError();
                if (st == RKSC_OK) st = RKSC_ERR_CUDA;
            }
        }
        {
            std::lock_guard<std::mutex> lock(p->mu);
            s.plan = plan;
            s.status = st;
            s.worker_done = true;
            p->next_attention = t + 1;
        }
        p->cv_turn.notify_all();
        p->cv_done.notify_all();
    }
}

void free_slot(Slot& s) {
    if (s.plan) rksc_plan_destroy(s.plan);
    if (s.map_dev) cudaFree(s.map_dev);
    if (s.sigma_dev) cudaFree(s.sigma_dev);
    if (s.status_dev) cudaFree(s.status_dev);
    if (s.map_host) cudaFreeHost(s.map_host);
    if (s.workspace) cudaFree(s.workspace);
    for (cudaEvent_t e : {s.ev_map, s.ev_att, s.ev_done, s.ev_seg0, s.ev_seg1})
        if (e) cudaEventDestroy(e);
    s = Slot{};
}

}  // namespace

extern "C" RKSC_API void rksc_pipeline_destroy(rksc_pipeline* p) {
    if (!p) return;
    int cur = -1;
    const bool sw = p->device >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != p->device;
    if (sw) cudaSetDevice(p->device);
    {
        std::lock_guard<std::mutex> lock(p->mu);
        p->stop = true;
    }
    p->cv_jobs.notify_all();
    for (auto& w : p->workers)
        if (w.joinable()) w.join();   // workers finish the queued steps first
    if (p->gate_stream) cudaStreamSynchronize(p->gate_stream);
    if (p->att_stream) cudaStreamSynchronize(p->att_stream);
    if (p->copy_stream) cudaStreamSynchronize(p->copy_stream);
    for (auto& s : p->slots) free_slot(s);
    if (p->ev_inputs) cudaEventDestroy(p->ev_inputs);
    if (p->gate_stream) cudaStreamDestroy(p->gate_stream);
    if (p->att_stream) cudaStreamDestroy(p->att_stream);
    if (p->copy_stream) cudaStreamDestroy(p->copy_stream);
    cudaGetLastError();
    if (sw) cudaSetDevice(cur);
    delete p;
}

extern "C" RKSC_API int32_t rksc_pipeline_create(const rksc_layout* layout, int32_t B, int32_t P, int32_t L, int32_t D,
                                                 float alpha, float tau, const int32_t* shared_off,
                                                 const int32_t* shared_pages, const int32_t* shared_ntok,
                                                 const int32_t* priv_off, const int32_t* priv_pages,
                                                 const int32_t* priv_ntok, const int32_t* sfx_off,
                                                 const int32_t* sfx_pages, const int32_t* sfx_ntok, int32_t depth,
                                                 int64_t mass_capacity, int32_t timing, rksc_pipeline** out) {
    if (!out) return RKSC_ERR_INVALID_ARG;
    *out = nullptr;
    if (!layout || B <= 0 || P <= 0 || L <= 0 || D <= 0 || depth < 2 || depth > 8 || mass_capacity < 0)
        return RKSC_ERR_INVALID_ARG;
    if (!shared_off || !shared_ntok || !priv_off || !priv_ntok || !sfx_off || !sfx_ntok) return RKSC_ERR_INVALID_ARG;
    if ((shared_off[P] > 0 && !shared_pages) || (priv_off[B] > 0 && !priv_pages) || (sfx_off[B] > 0 && !sfx_pages))
        return RKSC_ERR_INVALID_ARG;
    rksc_pipeline* p = new (std::nothrow) rksc_pipeline();
    if (!p) return RKSC_ERR_NOMEM;
    try {
        p->lists[0].assign(shared_off, shared_off + P + 1);
        p->lists[1].assign(shared_pages, shared_pages + (shared_off[P] > 0 ? shared_off[P] : 0));
        p->lists[2].assign(shared_ntok, shared_ntok + P);
        p->lists[3].assign(priv_off, priv_off + B + 1);
        p->lists[4].assign(priv_pages, priv_pages + (priv_off[B] > 0 ? priv_off[B] : 0));
        p->lists[5].assign(priv_ntok, priv_ntok + B);
        p->lists[6].assign(sfx_off, sfx_off + B + 1);
        p->lists[7].assign(sfx_pages, sfx_pages + (sfx_off[B] > 0 ? sfx_off[B] : 0));
        p->lists[8].assign(sfx_ntok, sfx_ntok + B);
        for (auto& v : p->lists)
            if (v.empty()) v.push_back(0);   // data() of an empty list must still be a pointer
        p->slots.resize(depth);
    } catch (const std::bad_alloc&) {
        delete p;
        return RKSC_ERR_NOMEM;
    }
    p->layout = *layout;
    p->B = B;
    p->P = P;
    p->L = L;
    p->D = D;
    p->alpha = alpha;
    p->tau = tau;
    p->depth = depth;
    p->mass_capacity = mass_capacity;
    p->timing = timing > 0 ? timing : 0;
    bool ok = cudaGetDevice(&p->device) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&p->gate_stream, cudaStreamNonBlocking) == cudaSuccess;
    // the attention stream outranks the gate stream: where both have thread blocks waiting for an SM,
    // the persistent attention kernels get it, and the gates of later steps fill what is left
    int prio_lo = 0, prio_hi = 0;
    ok = ok && cudaDeviceGetStreamPriorityRange(&prio_lo, &prio_hi) == cudaSuccess;
    ok = ok && cudaStreamCreateWithPriority(&p->att_stream, cudaStreamNonBlocking, prio_hi) == cudaSuccess;
    ok = ok && cudaStreamCreateWithFlags(&p->copy_stream, cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&p->ev_inputs, cudaEventDisableTiming) == cudaSuccess;
    for (auto& s : p->slots) {
        ok = ok && cudaMalloc(reinterpret_cast<void**>(&s.map_dev), (size_t)B * 4) == cudaSuccess;
        ok = ok && cudaMalloc(reinterpret_cast<void**>(&s.sigma_dev), (size_t)B * 4) == cudaSuccess;
        ok = ok && cudaMalloc(reinterpret_cast<void**>(&s.status_dev), 16) == cudaSuccess;
        ok = ok && cudaMallocHost(reinterpret_cast<void**>(&s.map_host), (2 * (size_t)B + 4) * 4) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&s.ev_map, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&s.ev_att, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&s.ev_done, cudaEventDisableTiming) == cudaSuccess;
        if (p->timing > 0) {
            ok = ok && cudaEventCreate(&s.ev_seg0) == cudaSuccess;
            ok = ok && cudaEventCreate(&s.ev_seg1) == cudaSuccess;
        }
    }
    if (!ok) {
        cudaGetLastError();
        rksc_pipeline_destroy(p);
        return RKSC_ERR_CUDA;
    }
    try {
        const int nworkers = depth > 2 ? depth - 2 : 1;
        for (int i = 0; i < nworkers; ++i) p->workers.emplace_back(worker_main, p);
    } catch (...) {
        rksc_pipeline_destroy(p);
        return RKSC_ERR_NOMEM;
    }
    *out = p;
    return RKSC_OK;
}

extern "C" RKSC_API int32_t rksc_pipeline_submit(rksc_pipeline* p, const float* h_branch, const float* h_root,
                                                 const int32_t* cand_prefix, const void* q, const void* k_pool,
                                                 const void* v_pool, float* out, float* block_mass, void* after_stream,
                                                 int64_t* ticket) {
    if (!p || !h_branch || !h_root || !cand_prefix || !q || !k_pool || !v_pool || !out || !ticket)
        return RKSC_ERR_INVALID_ARG;
    const int64_t t = p->next_ticket;
    Slot& s = p->slots[t % p->depth];
    if (t >= p->depth) {
        // the slot's previous step must have been waited for (its outputs are the caller's to read first)
        if (!s.waited) return RKSC_ERR_INVALID_ARG;
    }
    if (s.plan) {
        rksc_plan_destroy(s.plan);
        s.plan = nullptr;
    }
    if (after_stream) {
        cudaStream_t us = static_cast<cudaStream_t>(after_stream);
        if (cudaEventRecord(p->ev_inputs, us) != cudaSuccess || cudaStreamWaitEvent(p->gate_stream, p->ev_inputs, 0) != cudaSuccess ||
            cudaStreamWaitEvent(p->att_stream, p->ev_inputs, 0) != cudaSuccess) {
            cudaGetLastError();
            return RKSC_ERR_CUDA;
        }
    }
    s.h_branch = h_branch;
    s.h_root = h_root;
    s.cand = cand_prefix;
    s.q = q;
    s.k_pool = k_pool;
    s.v_pool = v_pool;
    s.out = out;
    s.block_mass = block_mass;
    s.ticket = t;
    s.attention_enqueued = false;
    s.timed = false;
    cudaStream_t gs = p->gate_stream;
    int32_t st = RKSC_OK;
    if (cudaMemsetAsync(s.status_dev, 0, 16, gs) != cudaSuccess) st = RKSC_ERR_CUDA;
    if (st == RKSC_OK)
        st = rksc_asks_gate(h_branch, h_root, cand_prefix, p->B, p->P, p->L, p->D, p->alpha, p->tau, s.map_dev, s.sigma_dev, gs);
    if (st == RKSC_OK &&
        (cudaMemcpyAsync(s.map_host, s.map_dev, (size_t)p->B * 4, cudaMemcpyDeviceToHost, gs) != cudaSuccess ||
         cudaMemcpyAsync(s.map_host + p->B, s.sigma_dev, (size_t)p->B * 4, cudaMemcpyDeviceToHost, gs) != cudaSuccess ||
         cudaEventRecord(s.ev_map, gs) != cudaSuccess)) {   // (the worker waits for this on the host before it
                                                            //  enqueues the attention, which reads the cleared status word)
        cudaGetLastError();
        st = RKSC_ERR_CUDA;
    }
    {
        std::lock_guard<std::mutex> lock(p->mu);
        s.status = st;   // a failed gate still takes its turn, so that the order of the others holds
        s.worker_done = false;
        s.waited = false;
        p->jobs.push_back(t);
    }
    p->cv_jobs.notify_one();
    p->next_ticket = t + 1;
    *ticket = t;
    return RKSC_OK;
}

extern "C" RKSC_API int32_t rksc_pipeline_wait(rksc_pipeline* p, int64_t ticket, int32_t* branch_to_prefix, float* sigma,
                                               int64_t* mass_off, rksc_plan_info* info, float* segment_ms) {
    if (!p) return RKSC_ERR_INVALID_ARG;
    if (ticket != p->next_wait || ticket >= p->next_ticket) return RKSC_ERR_INVALID_ARG;
    Slot& s = p->slots[ticket % p->depth];
    {
        std::unique_lock<std::mutex> lock(p->mu);
        p->cv_done.wait(lock, [&] { return s.worker_done; });
    }
    int32_t st = s.status;
    if (st == RKSC_OK || s.attention_enqueued) {
        if (cudaEventSynchronize(s.ev_done) != cudaSuccess) {
            cudaGetLastError();
            if (st == RKSC_OK) st = RKSC_ERR_CUDA;
        }
    } else {
        // the step stopped before its attention: its gate work may still be running
        cudaEventSynchronize(s.ev_map);
        cudaGetLastError();
    }
    if (st == RKSC_OK) {
        const int32_t dev_status = s.map_host[2 * (size_t)p->B];
        if (dev_status != 0) st = dev_status;
    }
    if (st == RKSC_OK || st == RKSC_ERR_WORKSPACE || st == RKSC_ERR_DEVICE_TIMEOUT) {
        if (branch_to_prefix) std::memcpy(branch_to_prefix, s.map_host, (size_t)p->B * 4);
        if (sigma) std::memcpy(sigma, s.map_host + p->B, (size_t)p->B * 4);
    }
    if (s.plan) {
        rksc_plan_info pi{};
        if (rksc_plan_query(s.plan, &pi) == RKSC_OK) {
            if (info) *info = pi;
            if (mass_off && pi.mass_off) std::memcpy(mass_off, pi.mass_off, ((size_t)p->B + 1) * sizeof(int64_t));
            if (info) info->mass_off = nullptr;   // the plan is the pipeline's and does not outlive the slot
        }
    }
    if (segment_ms) {
        *segment_ms = 0.f;
        if (s.timed && s.attention_enqueued && cudaEventElapsedTime(segment_ms, s.ev_seg0, s.ev_seg1) != cudaSuccess)
            cudaGetLastError();
    }
    s.waited = true;
    p->next_wait = ticket + 1;
    return st;
}
