#!/usr/bin/env python
"""Benchmark of the ASKS hot path on B200: gate -> tables -> plan -> shared-prefix decode attention.

One "step" is one pass of the whole path over one batch of synthetic input that is already in
HBM: the gate kernel, the map's copy to the host, table and plan construction, and the
branch-decode attention (segment kernel + merge).  The metric is unique-KV bytes per second:
the valid tokens of the distinct KV segments the batch references, times bytes per token,
divided by the step time.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

Prints one JSON line (rank 0).  With N > 1 (launched by torchrun) every rank runs its own
batch (seed + rank): the path shards by problem, there is no collective on the data path.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

METRIC = "branch_decode_attention_unique_kv_throughput"
UNIT = "TB/s"
NOMINAL_HBM_TBPS = 8.0       # the figure the target (>= 70 %) is stated against
FALLBACK_HBM_GBS = 6650.0    # used only when MEASURED_PEAKS.json is absent

# dram__bytes_read.sum + dram__bytes_write.sum of one launch of the segment kernel, from the ncu
# capture summarised under profiles/ (None until a capture of that workload exists).
NCU_TRAFFIC_BYTES = {"batched_serving": 767356672}   # profiles/seg_attention_batched_serving.md

WORKLOAD_LABEL = {
    "tiny": "configs[0] tiny: 8q/2kv d64, 4 branches, prefix 256 + suffix 32",
    "qwen_layer": "configs[1] Qwen-7B-shaped layer: 28q/4kv d128, 4 branches, prefix 2048 + suffix 512",
    "tot": "configs[2] Tree-of-Thoughts (4,3): 64 leaves, root 1024 + 3 x 256, 32q/8kv d128",
    "batched_serving": "configs[3] batched serving: 32 problems x 8 branches, prefix U[512,4096], "
                       "suffix U[128,1024], 28q/4kv d128, 30% of branches below tau",
    "long_context": "configs[4] long context with eviction holes: 16 branches, prefix 32768 (20% of pages "
                    "evicted) + suffix 2048, 32q/8kv d128",
    "diverse_phrasing": "diverse-phrasing regime (an extra workload beside the five configurations): 15 problems x 8 phrasings at 4 divergence "
                        "levels, prefix 512, suffix U[16,144], 28q/4kv d128, alpha 1.5, tau 0.82; the gate shares "
                        "the identical and the minor-rewording phrasings",
    "long_prefix_serving": "batched serving with long prefixes (an extra workload beside the five configurations): 32 "
                           "problems x 8 branches, prefix U[4096,16384], suffix U[16,128], 28q/4kv d128, 30% of "
                           "branches below tau",
}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="batched_serving", choices=list(WORKLOAD_LABEL))
    ap.add_argument("--cpu-sample-branches", type=int, default=0, help="branches the oracle runs (0 = the whole batch)")
    ap.add_argument("--e2e-steps", type=int, default=10)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sweep", action="store_true", help="skip the per-config attention-only table")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-pipeline", action="store_true", help="time the steps strictly one after another")
    ap.add_argument("--pipeline-depth", type=int, default=4,
                    help="steps the library's pipeline keeps in flight in the headline loop (2..8; depth - 2 host threads)")
    ap.add_argument("--cgee-only", action="store_true",
                    help="run only the CGEE entropy-kernel measurement and print its object (used for profiling)")
    ap.add_argument("--model-step-only", action="store_true",
                    help="run only the whole-model decode-step measurement (all layers, eager and as a CUDA graph)")
    return ap.parse_args()


def measured_peak_gbs():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------------------
# clocks sampling during the timed region
# ----------------------------------------------------------------------------------------------

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML from a thread while the timed region runs."""

    REASONS = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
               "hw_thermal_slowdown": 0x40, "hw_power_brake_slowdown": 0x80}

    def __init__(self, torch_device):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self._nv = pynvml
            uuid = getattr(torch.cuda.get_device_properties(torch_device), "uuid", None)
            try:
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(torch_device.index or 0)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _run(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(float(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                try:
                    mask = nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)
                except Exception:
                    mask = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for name, bit in self.REASONS.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def start(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join(timeout=2)
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ----------------------------------------------------------------------------------------------
# workload set-up
# ----------------------------------------------------------------------------------------------

def load_workload(name: str, seed_shift: int = 0):
    import workloads
    base = {"tiny": 0, "qwen_layer": 1, "tot": 2, "batched_serving": 3, "long_context": 4,
            "diverse_phrasing": 5, "long_prefix_serving": 6}[name]
    return workloads.make_config(name, seed=workloads.generators.SEED_BASE + base + 1000 * seed_shift)


class DeviceBatch:
    """A workload resident in HBM plus the reusable output buffers."""

    def __init__(self, w, dev):
        import torch
        self.w = w
        self.dev = dev
        self.q = w.q.to(dev)
        self.k_pool = w.k_pool.to(dev)
        self.v_pool = w.v_pool.to(dev)
        self.has_gate = w.gate is not None and w.flat is not None
        if w.gate is not None:
            self.h_branch = w.gate.h_branch.to(dev)
            self.h_root = w.gate.h_root.to(dev)
            self.cand = torch.from_numpy(w.gate.cand_prefix).to(dev)
            self.map_dev = torch.empty(self.q.shape[0], dtype=torch.int32, device=dev)
            self.sigma_dev = torch.empty(self.q.shape[0], dtype=torch.float32, device=dev)
            self.map_host = torch.empty(self.q.shape[0], dtype=torch.int32).pin_memory()
        self.status = torch.zeros(1, dtype=torch.int32, device=dev)
        self.out = torch.empty(tuple(self.q.shape), dtype=torch.float32, device=dev)
        self.mass = None
        self.workspace = None
        self.tables = None
        import paper_2606_09937_b200 as rk
        self.layout = rk.Layout.of(w.layout)
        self.lists = rk.GateLists(w.flat) if self.has_gate else None
        if w.tables is not None:
            self.tables = rk.Tables.of(w.tables)

    def ensure_buffers(self, plan):
        import torch
        if self.mass is None or self.mass.numel() < max(plan.mass_elems, 1):
            self.mass = torch.empty(max(plan.mass_elems, 1), dtype=torch.float32, device=self.dev)
        if self.workspace is None or self.workspace.numel() < plan.workspace_bytes:
            self.workspace = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=self.dev)


def run_step(rk, batch: DeviceBatch, seg_events=None):
    """One pass of the hot path.  Returns the plan (for byte counts) and the number of kernel launches
    (gate, tcgen05 segment kernel, warp segment kernel, merge; the plan knows which it needs)."""
    w = batch.w
    launches = 0
    if batch.has_gate:
        g, f = w.gate, w.flat
        rk.rksc_asks_gate(batch.h_branch, batch.h_root, batch.cand, g.alpha, g.tau,
                          branch_to_prefix=batch.map_dev, sigma=batch.sigma_dev)
        launches += 1
        batch.map_host.copy_(batch.map_dev, non_blocking=False)   # the host needs the map to build tables
        plan = rk.rksc_plan_create_from_gate(batch.layout, batch.map_host.numpy(), batch.lists)
    else:
        plan = rk.rksc_plan_create(batch.layout, batch.tables)
    batch.ensure_buffers(plan)
    kw = dict(out=batch.out, block_mass=batch.mass, workspace=batch.workspace, device_status=batch.status)
    if seg_events is None:
        rk.rksc_branch_decode_attention(plan, batch.q, batch.k_pool, batch.v_pool, **kw)
    else:
        seg_events[0].record()
        rk.rksc_branch_decode_attention(plan, batch.q, batch.k_pool, batch.v_pool, phases=1, **kw)
        seg_events[1].record()
        rk.rksc_branch_decode_attention(plan, batch.q, batch.k_pool, batch.v_pool, phases=2, **kw)
    launches += plan.num_kernel_launches
    return plan, launches


def attention_only_times(rk, batch: DeviceBatch, plan, iters: int, flush):
    """Per-iteration CUDA-event times (ms) of the attention call alone, L2 flushed before each."""
    import torch
    kw = dict(out=batch.out, block_mass=batch.mass, workspace=batch.workspace, device_status=batch.status)
    times = []
    for _ in range(iters):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rk.rksc_branch_decode_attention(plan, batch.q, batch.k_pool, batch.v_pool, **kw)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    return times


def algorithmic_bytes(plan, layout):
    """Bytes the segment kernel has to move by definition: unique KV + queries + page ids + block masses."""
    bpt = 2 * layout.num_kv_heads * layout.head_dim * 2
    kv = plan.unique_kv_tokens * bpt
    qb = plan.num_branches * layout.num_q_heads * layout.head_dim * 2
    tables = 4 * plan.num_pages_listed
    mass = 4 * plan.mass_elems
    return kv, kv + qb + tables + mass


# ----------------------------------------------------------------------------------------------
# the oracle as CPU baseline / reference arm
# ----------------------------------------------------------------------------------------------

def oracle_pass(w, sample_branches: int):
    """The oracle on a bounded sample (the first branches of the batch).  Returns (seconds, unique bytes, cores)."""
    import oracle
    import workloads
    try:
        from threadpoolctl import threadpool_info
        cores = max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        cores = 1
    L = w.layout
    q = oracle.to_f32_numpy(w.q)
    kp = oracle.to_f32_numpy(w.k_pool)
    vp = oracle.to_f32_numpy(w.v_pool)
    t0 = time.perf_counter()
    if w.gate is not None and w.flat is not None:
        g, f = w.gate, w.flat
        m, _ = oracle.asks_gate(g.h_branch.numpy(), g.h_root.numpy(), g.cand_prefix, g.alpha, g.tau)
        t = oracle.tables_from_gate(m, f.num_prefixes, f.shared_off, f.shared_pages, f.shared_ntok,
                                    f.priv_off, f.priv_pages, f.priv_ntok, f.sfx_off, f.sfx_pages, f.sfx_ntok)
    else:
        tt = w.tables
        t = {k: getattr(tt, k) for k in ("seg_block_off", "seg_blocks", "seg_num_tokens", "br_seg_off", "br_segs")}
    B = len(t["br_seg_off"]) - 1
    nb = B if sample_branches <= 0 else min(B, sample_branches)
    oracle.branch_decode_attention(L.num_q_heads, L.num_kv_heads, L.head_dim, L.sm_scale,
                                   t["seg_block_off"], t["seg_blocks"], t["seg_num_tokens"],
                                   t["br_seg_off"], t["br_segs"], q, kp, vp, branches=range(nb))
    dt = time.perf_counter() - t0
    segs = np.unique(t["br_segs"][: t["br_seg_off"][nb]])
    ubytes = int(sum(int(t["seg_num_tokens"][s]) for s in segs)) * L.bytes_per_token
    return dt, ubytes, cores, nb, B


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = load_workload(args.workload)
    times, ub = [], 0
    nb = B = 0
    cores = 1
    for i in range(args.warmup + args.steps):
        dt, ub, cores, nb, B = oracle_pass(w, args.cpu_sample_branches)
        if i >= args.warmup:
            times.append(dt)
    t = sum(times) / len(times)
    val = ub / t / 1e12
    sample = f"{nb} of {B} branches of the batch per step (gate over all branches, attention over these)"
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOAD_LABEL[args.workload], "sample": sample},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


# ----------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import paper_2606_09937_b200 as rk

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the library has no CPU path")
    rk.lib()
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    l2_bytes = torch.cuda.get_device_properties(dev).L2_cache_size
    flush_buf = torch.empty(max(2 * l2_bytes, 256 << 20), dtype=torch.uint8, device=dev)

    def flush():
        flush_buf.fill_(1)

    if args.cgee_only:
        if rank == 0:
            print(json.dumps({"cgee": cgee_measurement(rk, dev, flush, measured_peak_gbs()[0], iters=max(3, args.steps))}))
        return

    if args.model_step_only:
        if rank == 0:
            print(json.dumps({"model_step": model_step_measurement(rk, dev, args.workload)}))
        return

    w = load_workload(args.workload, seed_shift=rank)
    batch = DeviceBatch(w, dev)
    if w.name == "long_context":
        punch_long_context(rk, batch)

    plan = None
    for _ in range(max(args.warmup, 3)):
        plan, _ = run_step(rk, batch)
    torch.cuda.synchronize()
    assert int(batch.status.item()) == 0, "a kernel reported a device-side timeout"
    kv_bytes, alg_bytes = algorithmic_bytes(plan, w.layout)
    small = kv_bytes < 2 * l2_bytes   # then L2 must be flushed between timed iterations

    sampler = ClockSampler(dev)
    if rank == 0:
        sampler.start()
    seg_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    step_ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    launches = 0
    barrier()
    t_wall0 = time.perf_counter()
    for i in range(args.steps):
        if small:
            flush()
        step_ev[i][0].record()
        plan, n = run_step(rk, batch, seg_events=seg_ev[i])
        step_ev[i][1].record()
        launches += n
    barrier()
    t_wall = time.perf_counter() - t_wall0
    step_ms = [a.elapsed_time(b) for a, b in step_ev]
    seg_ms = [a.elapsed_time(b) for a, b in seg_ev]
    total_ms = sum(step_ms)           # device time of exactly K steps (flushes excluded)
    assert int(batch.status.item()) == 0, "a kernel reported a device-side timeout"
    serial = {"ms_per_step": total_ms / args.steps, "wall_ms_per_step": t_wall * 1e3 / args.steps,
              "tbps_unique_kv": kv_bytes * args.steps / (total_ms * 1e-3) / 1e12,
              "what": "the same K steps strictly one after another on one stream"}
    pipelined = batch.has_gate and not small and not args.no_pipeline
    if pipelined:
        # the headline loop: the library's step pipeline (rksc_pipeline_*) keeps `depth` whole steps in flight on
        # its own gate stream, attention stream and host threads; this thread only submits and waits
        depth = max(2, min(8, args.pipeline_depth))
        g, f = w.gate, w.flat
        B = w.num_branches
        cap = 0
        for b in range(B):
            r = int(g.cand_prefix[b])
            cap += max(int(f.shared_off[r + 1] - f.shared_off[r]), int(f.priv_off[b + 1] - f.priv_off[b]))
            cap += int(f.sfx_off[b + 1] - f.sfx_off[b])
        cap *= w.layout.num_q_heads                      # block masses of a step whatever its gate map
        pipe = rk.Pipeline(batch.layout, B, tuple(g.h_branch.shape[1:]), g.alpha, g.tau, batch.lists, depth=depth,
                           mass_capacity=cap, timing=4)       # events around the segment kernels of every 4th step
        bufs = [(torch.empty_like(batch.out), torch.empty(cap, dtype=torch.float32, device=dev)) for _ in range(depth)]
        ticket = [0]

        def run_pipeline(nsteps, after=None):
            """Submits nsteps steps, never more than `depth` in flight; returns their results."""
            res, first = [], ticket[0]
            for i in range(nsteps):
                t = ticket[0]
                if t - first >= depth:
                    res.append(pipe.wait(t - depth))
                o, m = bufs[t % depth]
                pipe.submit(batch.h_branch, batch.h_root, batch.cand, batch.q, batch.k_pool, batch.v_pool, o, m,
                            after_stream=after if i == 0 else None)
                ticket[0] = t + 1
            for t in range(max(first, ticket[0] - depth), ticket[0]):
                res.append(pipe.wait(t))
            return res

        run_pipeline(max(args.warmup, 3) + 2 * depth)         # untimed warm-up
        torch.cuda.synchronize()
        e_start, e_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        t_wall0 = time.perf_counter()
        e_start.record()
        # the first step waits for e_start through `after`; the last wait returns when the last step has finished
        results = run_pipeline(args.steps, after=torch.cuda.current_stream())
        e_end.record()
        barrier()
        t_wall = time.perf_counter() - t_wall0
        total_ms = e_start.elapsed_time(e_end)
        assert len(results) == args.steps and all(r.status == 0 for r in results)
        seg_ms = [r.segment_ms for r in results if r.segment_ms > 0.0]
        launches = sum(1 + r.num_kernel_launches for r in results)
        assert all(np.array_equal(r.branch_to_prefix, batch.map_host.numpy()) for r in results[:3])
        pipe.close()
        del bufs
    clocks = sampler.stop() if rank == 0 else None
    value, total_ms_max = aggregate_over_ranks(dist, dev, kv_bytes, args.steps, total_ms)
    peak_gbs, peak_kind = measured_peak_gbs()
    seg_avg_ms = sum(seg_ms) / len(seg_ms)
    achieved = alg_bytes / (seg_avg_ms * 1e-3) / 1e9
    B = w.num_branches

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms_max / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {
            "workload": WORKLOAD_LABEL[args.workload],
            "step": "gate kernel + map D2H + tables + plan + attention (segment kernels + merge)",
            "pipelining": (f"rksc_pipeline, {depth} steps in flight: one gate stream, one attention stream (attention "
                           f"launches back to back in step order, the gates of later steps beside them) and "
                           f"{max(1, depth - 2)} host thread(s) of the library that build tables and plans; CUDA events "
                           f"around the segment kernels of every 4th step") if pipelined
            else "none (steps strictly serial)",
            "unique_kv_bytes": kv_bytes, "branches": B, "work_items": plan.num_work_items,
            "l2": ("inputs larger than L2 (unique KV %.0f MB vs L2 %.0f MB)" % (kv_bytes / 1e6, l2_bytes / 1e6))
            if not small else "L2 flushed (write of 2x L2) before every timed step",
            "sharding": "one batch per rank (seed + rank), no data-path collective",
        },
        "branch_steps_per_s": world * B * args.steps / (total_ms_max * 1e-3),
        "pct_of_8tbps": 100.0 * value / world / NOMINAL_HBM_TBPS,
        "pct_of_measured_copy_peak": 100.0 * value * 1e3 / world / peak_gbs,
        "wall_ms_per_step": t_wall * 1e3 / args.steps,
        "gpu_launches": launches,
        "serial_steps": serial,
        "roofline": {
            "kernel": "segment attention: seg_attn_tc_kernel + seg_attn_warp_kernel (chained launches)", "bound": "hbm", "achieved": achieved, "peak": peak_gbs,
            "unit": "GB/s", "frac": achieved / peak_gbs, "peak_source": peak_kind,
            "algorithmic_bytes_per_launch": alg_bytes, "avg_launch_ms": seg_avg_ms,
            "traffic": NCU_TRAFFIC_BYTES.get(args.workload),
        },
        "clocks": clocks,
        "paper_context": {"what": "the paper's own end-to-end speed-ups of its whole system (single A100, PyTorch SDPA, "
                                  "its datasets and models): context only, not comparable with a kernel throughput",
                          "mean_speedup_over_no_kv": 3.008, "speedup_over_prefix_caching": 1.66},
    }

    if rank == 0 and world == 1:
        att = attention_only_times(rk, batch, plan, max(10, args.steps), flush)
        med = statistics.median(att)
        line["attention_only"] = {
            "what": "one rksc_branch_decode_attention call (segment kernel + merge), plan prebuilt, cold L2",
            "ms_median": med, "ms_min": min(att), "tbps_unique_kv": kv_bytes / (med * 1e-3) / 1e12,
            "pct_of_8tbps": 100.0 * kv_bytes / (med * 1e-3) / 1e12 / NOMINAL_HBM_TBPS,
            "pct_of_measured_copy_peak": 100.0 * kv_bytes / (med * 1e-3) / 1e9 / peak_gbs,
            "branch_steps_per_s": B / (med * 1e-3),
        }
        # RSBCM (Section 2.4, Algorithm 4) on this step's masses: every listed page competes, N_max = 2000
        _, info = rsbcm_pass(rk, batch, plan, batch.mass, slice(0, plan.num_pages_listed), 2000)
        info["what"] = ("after a step, outside the timed region: rksc_rsbcm_page_scores over the step's block masses, "
                        "then rksc_rsbcm_evict down to the paper's default capacity of 2000 entries")
        line["rsbcm"] = info
        if batch.has_gate:
            line["stages"] = stage_times(rk, batch, flush)
        if not args.no_e2e and batch.has_gate:
            line["e2e"] = run_e2e(rk, batch, kv_bytes, args.e2e_steps)
        if not args.no_sweep:
            line["configs"] = sweep_configs(rk, dev, flush, peak_gbs, skip=args.workload, cached=(args.workload, line))
            line["suffix_prefill"] = suffix_prefill_measurement(rk, dev, flush, args.workload, 16)
            line["cgee"] = cgee_measurement(rk, dev, flush, peak_gbs)
            line["decode_loop"] = decode_loop_measurement(rk, dev, args.workload)
            line["model_step"] = model_step_measurement(rk, dev, args.workload)
            ms_ = line["model_step"]
            line["configs"][args.workload]["replica_ring"] = {
                "us_per_call": ms_["graph_us_per_layer"], "replicas": ms_["layers"], "cold": True,
                "tbps_unique_kv": ms_["tbps_unique_kv"], "pct_of_8tbps": ms_["pct_of_8tbps"]}
            iso_ms = line["model_step"]["segment_kernels_us_per_layer"] * 1e-3
            line["roofline"]["isolated"] = {
                "what": "the same two kernels with nothing beside them: 28 layers' segment launches replayed back to back "
                        "as one CUDA graph, every layer on its own cold pool (model_step); the figures above are taken "
                        "inside the pipelined loop, where the gate kernels of later steps run beside them",
                "avg_launch_ms": iso_ms, "achieved": alg_bytes / (iso_ms * 1e-3) / 1e9,
                "frac": alg_bytes / (iso_ms * 1e-3) / 1e9 / peak_gbs}
        if not args.no_cpu_baseline:
            # about 10-30 s of oracle work: whole passes over the batch until 10 s have gone by
            passes, total, ub, cores, nb, Bt = 0, 0.0, 0, 1, 0, 0
            while total < 10.0 and passes < 8:
                dt, ub, cores, nb, Bt = oracle_pass(w, args.cpu_sample_branches)
                total += dt
                passes += 1
            line["cpu_baseline"] = {
                "value": ub * passes / total / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle",
                "sample": f"{nb} of {Bt} branches of the batch (gate over all branches, attention over these), "
                          f"{passes} passes, {total:.1f} s in all", "seconds": total}
    if rank == 0:
        print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def run_e2e(rk, batch: DeviceBatch, kv_bytes: int, steps: int):
    """The metric through rksc_decode_step_host: per-step inputs in pinned host memory, results read back.

    The KV pool stays resident (it is device state written by earlier decode steps); hidden states,
    candidate ids, page lists and queries go host -> device and map, sigma, out and block masses come
    back inside every timed step."""
    import torch
    w = batch.w
    g, L = w.gate, w.layout
    B = w.num_branches
    hb = g.h_branch.pin_memory()
    hr = g.h_root.pin_memory()
    q = w.q.pin_memory()
    m_host = torch.empty(B, dtype=torch.int32).pin_memory()
    s_host = torch.empty(B, dtype=torch.float32).pin_memory()
    out_host = torch.empty((B, L.num_q_heads, L.head_dim), dtype=torch.float32).pin_memory()
    mass_host = torch.empty(max(batch.mass.numel(), 1), dtype=torch.float32).pin_memory()
    mass_off = np.zeros(B + 1, dtype=np.int64)

    def one():
        rk.rksc_decode_step_host(L, hb, hr, g.cand_prefix, g.alpha, g.tau, w.flat, q, batch.k_pool, batch.v_pool,
                                 m_host, s_host, out_host, mass_host, mass_off)
    for _ in range(3):
        one()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    for _ in range(steps):
        one()
    e1.record()
    e1.synchronize()
    wall = time.perf_counter() - t0
    ms = e0.elapsed_time(e1) / steps
    mass_elems = int(mass_off[-1]) * L.num_q_heads
    h2d = hb.numel() * 4 + hr.numel() * 4 + B * 4 + q.numel() * 2
    d2h = B * 4 * 2 + out_host.numel() * 4 + mass_elems * 4 + 4
    return {"value": kv_bytes / (ms * 1e-3) / 1e12, "unit": UNIT, "h2d_bytes_per_step": int(h2d),
            "d2h_bytes_per_step": int(d2h), "ms_per_step": ms, "wall_ms_per_step": wall * 1e3 / steps,
            "call": "rksc_decode_step_host (pinned host buffers; KV pool resident in HBM)", "steps": steps}


def aggregate_over_ranks(dist, dev, kv_bytes: int, steps: int, total_ms: float):
    """Whole-job throughput: bytes summed over ranks (each rank has its own batch), time = max over ranks."""
    import torch
    t = torch.tensor([total_ms], dtype=torch.float64, device=dev)
    b = torch.tensor([float(kv_bytes)], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        dist.all_reduce(b, op=dist.ReduceOp.SUM)
    total_ms_max = float(t.item())
    return float(b.item()) * steps / (total_ms_max * 1e-3) / 1e12, total_ms_max


def _event_us(fn, iters=20):
    import torch
    for _ in range(3):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) * 1e3 / iters


def stage_times(rk, batch: "DeviceBatch", flush, iters: int = 12):
    """The stages of a step one by one, outside the timed region: the gate kernel (device time after a
    write-flush of L2), the copy of its map to the host, and tables + plan on the host (wall time of
    rksc_plan_create_from_gate, which ends with the upload of the plan's arrays)."""
    import torch
    g = batch.w.gate
    gate_us, copy_us, plan_us = [], [], []
    for _ in range(iters):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rk.rksc_asks_gate(batch.h_branch, batch.h_root, batch.cand, g.alpha, g.tau,
                          branch_to_prefix=batch.map_dev, sigma=batch.sigma_dev)
        e1.record()
        e1.synchronize()
        gate_us.append(e0.elapsed_time(e1) * 1e3)
        t0 = time.perf_counter()
        batch.map_host.copy_(batch.map_dev, non_blocking=False)
        t1 = time.perf_counter()
        plan = rk.rksc_plan_create_from_gate(batch.layout, batch.map_host.numpy(), batch.lists)
        t2 = time.perf_counter()
        copy_us.append((t1 - t0) * 1e6)
        plan_us.append((t2 - t1) * 1e6)
        del plan
    med = lambda v: statistics.median(v[2:])
    gate_bytes = (batch.h_branch.numel() + batch.h_root.numel()) * 4
    return {"gate_kernel_us": med(gate_us), "gate_gbs": gate_bytes / (med(gate_us) * 1e-6) / 1e9,
            "gate_bytes": gate_bytes, "map_to_host_us": med(copy_us), "tables_and_plan_host_us": med(plan_us),
            "what": "each stage alone, outside the timed region: gate kernel after a write-flush of L2 (CUDA events), "
                    "blocking copy of the map (host wall time), rksc_plan_create_from_gate (host wall time)"}


def rsbcm_pass(rk, batch: DeviceBatch, plan, mass, entries: slice, capacity: int, timed: bool = True):
    """RSBCM on the masses of a finished step (Section 2.4, Algorithm 4), all on the GPU: page scores,
    then the eviction among `entries` (depth 0) down to `capacity`.  Returns (host mask over all the
    plan's entries, timing dict)."""
    import torch
    n_all = plan.num_pages_listed
    score = rk.rksc_rsbcm_page_scores(plan, mass)
    sub = score[entries]
    n = int(sub.numel())
    depth = torch.zeros(n, dtype=torch.int32, device=score.device)
    ev = torch.empty(n, dtype=torch.uint8, device=score.device)
    cnt = torch.empty(1, dtype=torch.int32, device=score.device)
    ws = torch.empty(rk.rksc_rsbcm_workspace_bytes(n), dtype=torch.uint8, device=score.device)
    rk.rksc_rsbcm_evict(sub, depth, capacity, ev, cnt, ws)
    torch.cuda.synchronize()
    mask = np.zeros(n_all, dtype=np.uint8)
    mask[entries] = ev.cpu().numpy()
    info = {"entries": n, "capacity": int(capacity), "evicted": int(cnt.item())}
    if timed:
        info["page_scores_us"] = _event_us(lambda: rk.rksc_rsbcm_page_scores(plan, mass, score))
        info["evict_us"] = _event_us(lambda: rk.rksc_rsbcm_evict(sub, depth, capacity, ev, cnt, ws))
    return mask, info


def punch_long_context(rk, batch: DeviceBatch):
    """Config 5: the 20 % of the prefix pages with the lowest attention mass of a prior full-table step are
    evicted - scores, selection and holed tables all by the library's RSBCM calls."""
    import torch
    import workloads
    w = batch.w
    plan = rk.rksc_plan_create(w.layout, w.tables)
    batch.ensure_buffers(plan)
    _, mass, _ = rk.rksc_branch_decode_attention(plan, batch.q, batch.k_pool, batch.v_pool, out=batch.out,
                                                 block_mass=batch.mass, workspace=batch.workspace,
                                                 device_status=batch.status)
    torch.cuda.synchronize()
    npg = int(w.tables.seg_block_off[1])
    mask, info = rsbcm_pass(rk, batch, plan, mass, slice(0, npg), npg - int(0.2 * npg))
    holed = rk.rksc_tables_drop_evicted(w.tables, mask)
    t = workloads.Tables(seg_block_off=holed.seg_block_off, seg_blocks=holed.seg_blocks,
                         seg_num_tokens=holed.seg_num_tokens, br_seg_off=holed.br_seg_off, br_segs=holed.br_segs)
    import dataclasses
    batch.w = dataclasses.replace(w, tables=t, flat=None)
    batch.tables = holed
    return info


def suffix_prefill_measurement(rk, dev, flush, workload: str, s: int):
    """Suffix prefill (Appendix "Stepwise Batched Decode", step 1) on a config's tables: the last s tokens of
    every branch's suffix attend causally on top of the shared cache, run as a decode attention over B * s
    virtual branches (rksc_tables_for_suffix_prefill).  Attention call alone, cold L2."""
    import torch
    w = load_workload(workload)
    b = DeviceBatch(w, dev)
    plan0, _ = run_step(rk, b)                     # the decode step's plan: the tables the gate gave
    torch.cuda.synchronize()
    if b.has_gate:
        f = w.flat
        t = rk.rksc_tables_from_gate(b.map_host.numpy(), f.num_prefixes, f.shared_off, f.shared_pages, f.shared_ntok,
                                     f.priv_off, f.priv_pages, f.priv_ntok, f.sfx_off, f.sfx_pages, f.sfx_ntok)
    else:
        t = b.tables
    vt = rk.rksc_tables_for_suffix_prefill(t, s)
    plan = rk.rksc_plan_create(b.layout, vt)
    B, Hq, d = b.q.shape
    g = torch.Generator(device="cpu").manual_seed(1234)
    q = torch.randn((B * s, Hq, d), generator=g, dtype=torch.float32).to(torch.bfloat16).to(dev)
    out = torch.empty((B * s, Hq, d), dtype=torch.float32, device=dev)
    mass = torch.empty(max(plan.mass_elems, 1), dtype=torch.float32, device=dev)
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    kw = dict(out=out, block_mass=mass, workspace=ws, device_status=b.status)
    times = []
    for _ in range(12):
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rk.rksc_branch_decode_attention(plan, q, b.k_pool, b.v_pool, **kw)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    assert int(b.status.item()) == 0
    med = statistics.median(times[2:])
    kv0, _ = algorithmic_bytes(plan0, b.w.layout)
    lay = b.w.layout
    flops = 4.0 * lay.head_dim * lay.num_q_heads * s * sum(
        int(t.seg_num_tokens[sg]) for bb in range(B) for sg in t.br_segs[t.br_seg_off[bb]:t.br_seg_off[bb + 1]])
    res = {"what": f"suffix prefill of s = {s} tokens per branch on {workload}: {B * s} virtual branches, "
                   "attention call alone (segment kernels + merge), plan prebuilt, cold L2",
           "ms_median": med, "query_tokens_per_s": B * s / (med * 1e-3),
           "unique_kv_bytes_of_the_decode_tables": kv0, "tbps_on_those_bytes": kv0 / (med * 1e-3) / 1e12,
           "kv_bytes_the_plan_reads": plan.unique_kv_tokens * 2 * lay.num_kv_heads * lay.head_dim * 2,
           "attention_tflops": flops / (med * 1e-3) / 1e12, "work_items": plan.num_work_items}
    del b
    torch.cuda.empty_cache()
    return res


def decode_loop_measurement(rk, dev, workload: str, steps: int = 32):
    """Token-by-token decode (Appendix "Stepwise Batched Decode", step 2) on a config's tables: every step
    appends one token per branch to the paged cache (tables on the host, keys and values on the device), builds
    the plan of the grown tables and runs the attention.  Strictly serial steps (each needs the previous token)."""
    import dataclasses
    import torch
    w = load_workload(workload)
    b = DeviceBatch(w, dev)
    run_step(rk, b)
    torch.cuda.synchronize()
    if b.has_gate:
        f = w.flat
        t = rk.rksc_tables_from_gate(b.map_host.numpy(), f.num_prefixes, f.shared_off, f.shared_pages, f.shared_ntok,
                                     f.priv_off, f.priv_pages, f.priv_ntok, f.sfx_off, f.sfx_pages, f.sfx_ntok)
    else:
        t = b.tables
    B, Hq, d = b.q.shape
    lay0 = w.layout
    extra = B * (steps // 16 + 2)
    nblk = lay0.num_pool_blocks
    grow = lambda p: torch.cat([p, torch.zeros((extra,) + tuple(p.shape[1:]), dtype=p.dtype, device=dev)])
    k_pool, v_pool = grow(b.k_pool), grow(b.v_pool)
    b.k_pool = b.v_pool = None
    lay = rk.Layout.of(dataclasses.replace(lay0, num_pool_blocks=nblk + extra))
    g = torch.Generator(device="cpu").manual_seed(77)
    k_new = torch.randn((B, lay0.num_kv_heads, d), generator=g).to(torch.bfloat16).to(dev)
    v_new = torch.randn((B, lay0.num_kv_heads, d), generator=g).to(torch.bfloat16).to(dev)
    # (page, slot) of every step: a pinned row per step (the host runs ahead of the GPU, so a row that was
    # reused would be overwritten before its copy has run) and one copy per step to the device
    Bp = (B + 3) // 4 * 4                                      # rows 16-byte aligned
    where_host = torch.empty((steps + 3, 2, Bp), dtype=torch.int32).pin_memory()
    where_np = where_host.numpy()
    where_dev = torch.empty((2, Bp), dtype=torch.int32, device=dev)
    new_pages = np.arange(nblk, nblk + B, dtype=np.int32)      # one spare page per branch per 16 steps
    plan = rk.rksc_plan_create(lay, t)
    out = torch.empty((B, Hq, d), dtype=torch.float32, device=dev)
    mass = torch.empty(max(plan.mass_elems, 1) + B * Hq * (steps // 16 + 2), dtype=torch.float32, device=dev)
    ws = torch.empty(2 * plan.workspace_bytes, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def one(step, t):
        t, page, slot = rk.rksc_tables_append_token(t, new_pages + B * (step // 16))
        where_np[step, 0, :B] = page
        where_np[step, 1, :B] = slot
        where_dev.copy_(where_host[step], non_blocking=True)
        rk.rksc_kv_append(lay, k_pool, v_pool, k_new, v_new, where_dev[0], where_dev[1])
        plan = rk.rksc_plan_create(lay, t)
        assert plan.workspace_bytes <= ws.numel() and plan.mass_elems <= mass.numel()
        rk.rksc_branch_decode_attention(plan, b.q, k_pool, v_pool, out=out, block_mass=mass, workspace=ws,
                                        device_status=status)
        return t, plan

    for step in range(3):                                    # warm-up steps (they grow the tables too)
        t, plan = one(step, t)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    for step in range(3, 3 + steps):
        t, plan = one(step, t)
    e1.record()
    e1.synchronize()
    wall = time.perf_counter() - t0
    assert int(status.item()) == 0
    ms = e0.elapsed_time(e1) / steps
    res = {"what": f"{steps} serial decode steps on {workload}: tables append (host) + keys/values append (device) + "
                   "plan of the grown tables + attention, one new token per branch and step",
           "ms_per_step": ms, "wall_ms_per_step": wall * 1e3 / steps, "tokens_per_s": B / (ms * 1e-3),
           "branches": B}
    del b
    torch.cuda.empty_cache()
    return res


def model_step_measurement(rk, dev, workload: str, layers: int = 28, iters: int = 5):
    """One decode step of a whole model: the attention of every layer, each layer on its own KV pool, all through
    the step's one plan (Appendix "Stepwise Batched Decode": the tables are the step's, not the layer's).  Timed
    twice: the calls enqueued one by one, and the same calls captured once in a CUDA graph and replayed.  The
    layers' pools together are far larger than L2, so every layer reads cold."""
    import dataclasses
    import torch
    import workloads
    w = load_workload(workload)
    b = DeviceBatch(w, dev)
    plan, _ = run_step(rk, b)
    torch.cuda.synchronize()
    B, Hq, d = b.q.shape
    kv_bytes, _ = algorithmic_bytes(plan, w.layout)
    base = dataclasses.replace(w, q=b.q, k_pool=b.k_pool, v_pool=b.v_pool)
    per_layer = [workloads.layer_variant(base, l) for l in range(layers)]
    outs = [torch.empty((B, Hq, d), dtype=torch.float32, device=dev) for _ in range(layers)]
    masses = [torch.empty(max(plan.mass_elems, 1), dtype=torch.float32, device=dev) for _ in range(layers)]
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)

    def enqueue(phases=3):
        for l, x in enumerate(per_layer):
            rk.rksc_branch_decode_attention(plan, x.q, x.k_pool, x.v_pool, out=outs[l], block_mass=masses[l],
                                            workspace=ws, device_status=status, phases=phases)

    def timed(fn):
        times, walls = [], []
        for _ in range(iters):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            t0 = time.perf_counter()
            e0.record()
            fn()
            walls.append(time.perf_counter() - t0)
            e1.record()
            e1.synchronize()
            times.append(e0.elapsed_time(e1))
        return statistics.median(times), statistics.median(walls) * 1e3

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        for _ in range(3):
            enqueue()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    eager_ms, eager_cpu_ms = timed(enqueue)
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        enqueue()
    graph.replay()
    torch.cuda.synchronize()
    graph_ms, graph_cpu_ms = timed(graph.replay)
    # the same without the merge: the two segment kernels alone, back to back on cold data, no other kernel
    # beside them - the launch duration the roofline object's "isolated" figures use
    seg_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(seg_graph):
        enqueue(phases=1)
    seg_graph.replay()
    torch.cuda.synchronize()
    seg_ms, _ = timed(seg_graph.replay)
    assert int(status.item()) == 0
    res = {"what": f"attention of {layers} layers of one decode step on {workload} (one plan, one pool per layer, "
                   f"{layers * kv_bytes / 1e9:.1f} GB of unique KV in all): enqueued call by call, and as one CUDA graph",
           "layers": layers, "graph_ms_per_step": graph_ms, "eager_ms_per_step": eager_ms,
           "graph_us_per_layer": graph_ms * 1e3 / layers,
           "segment_kernels_us_per_layer": seg_ms * 1e3 / layers,
           "graph_enqueue_cpu_ms": graph_cpu_ms, "eager_enqueue_cpu_ms": eager_cpu_ms,
           "tbps_unique_kv": layers * kv_bytes / (graph_ms * 1e-3) / 1e12,
           "pct_of_8tbps": 100.0 * layers * kv_bytes / (graph_ms * 1e-3) / 1e12 / NOMINAL_HBM_TBPS,
           "whole_model_branch_steps_per_s": B / (graph_ms * 1e-3)}
    del graph, seg_graph, per_layer, outs, masses, b
    torch.cuda.empty_cache()
    return res


def cgee_measurement(rk, dev, flush, peak_gbs, B=8, D=3584, V=152064, iters=12):
    """The entropy hook of CGEE (Section 2.3, Eq. 5 / Algorithm 3) on Qwen2.5-7B's shapes: B = 8 verify rows,
    D = 3584, V = 152064; synthetic W_u and hidden rows.  The kernel reads W_u once: HBM roofline on its bytes."""
    import torch
    import workloads
    h, w = workloads.make_cgee_inputs(B, D, V, seed=workloads.generators.SEED_BASE + 60)
    h, w = h.to(dev), w.to(dev)
    H = torch.empty(B, dtype=torch.float32, device=dev)
    P = torch.empty(B, dtype=torch.float32, device=dev)
    ws = torch.empty(int(rk.lib().rksc_cgee_workspace_bytes()), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    # Two copies of W_u (2.2 GB) read in turn, back to back: either is 8x the L2, so every call reads cold
    # without a flush (whose dirty lines would be written back underneath the timed call).
    w2 = w.clone()
    times = []
    for i in range(iters + 2):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rk.rksc_cgee_logit_entropy(h, w if i % 2 == 0 else w2, H, P, ws, status)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1))
    flushed = []
    for _ in range(4):                                     # for comparison: the same call after a write-flush
        flush()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        rk.rksc_cgee_logit_entropy(h, w, H, P, ws, status)
        e1.record()
        e1.synchronize()
        flushed.append(e0.elapsed_time(e1))
    assert int(status.item()) == 0
    Hp = torch.full((B,), float("inf"), dtype=torch.float32, device=dev)
    flags = rk.rksc_cgee_entropy_exit(H, Hp, 2, 2, 8.0, 3.0)
    torch.cuda.synchronize()
    med = statistics.median(times[2:])
    byts = V * D * 2 + B * D * 2
    res = {"what": f"rksc_cgee_logit_entropy: entropy and top-1 probability of softmax(h W_u^T), B = {B}, D = {D}, "
                   f"V = {V} (two launches: the fused kernel and a one-block merge); two copies of W_u read in turn, "
                   f"each 8x the L2 (inputs larger than L2, no flush)",
           "ms_median": med, "ms_after_write_flush": statistics.median(flushed), "w_u_bytes": V * D * 2,
           "roofline": {"bound": "hbm", "achieved": byts / (med * 1e-3) / 1e9, "peak": peak_gbs, "unit": "GB/s",
                        "frac": byts / (med * 1e-3) / 1e9 / peak_gbs, "algorithmic_bytes_per_launch": byts},
           "tflops": 2.0 * B * D * V / (med * 1e-3) / 1e12,
           "entropy_nats_min_max": [float(H.min()), float(H.max())], "exit_flags_at_first_layer": int(flags.sum())}
    del w2
    return res


L2_BYTES = 126 << 20


def replica_ring_us(rk, b: "DeviceBatch", plan, kv_bytes: int, max_replicas: int = 48, iters: int = 6):
    """Attention time per call when calls follow each other over a ring of R replicas of the pools (the layers
    of a model: same tables and plan, other values), captured once in a CUDA graph and replayed: R x unique
    KV >= 3 x L2 where R <= max_replicas allows it, so that every call reads cold without a flush in between
    (a write-flush leaves dirty lines that are written back underneath the timed call)."""
    import dataclasses
    import torch
    import workloads
    R = int(min(max_replicas, max(3, -(-3 * L2_BYTES // max(kv_bytes, 1)))))
    base = dataclasses.replace(b.w, q=b.q, k_pool=b.k_pool, v_pool=b.v_pool)
    ring = [workloads.layer_variant(base, l) for l in range(R)]
    kw = dict(out=b.out, block_mass=b.mass, workspace=b.workspace, device_status=b.status)

    def enqueue():
        for x in ring:
            rk.rksc_branch_decode_attention(plan, x.q, x.k_pool, x.v_pool, **kw)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        enqueue()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        enqueue()
    times = []
    for _ in range(iters):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        graph.replay()
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3 / R)
    assert int(b.status.item()) == 0
    us = statistics.median(times[1:])
    del graph, ring
    return {"us_per_call": us, "replicas": R, "cold": bool(R * kv_bytes >= 3 * L2_BYTES),
            "tbps_unique_kv": kv_bytes / (us * 1e-6) / 1e12,
            "pct_of_8tbps": 100.0 * kv_bytes / (us * 1e-6) / 1e12 / NOMINAL_HBM_TBPS}


def sweep_configs(rk, dev, flush, peak_gbs, skip, cached):
    """Attention-only time of every config (plan prebuilt), as context for the headline workload: one call after
    a write-flush of L2 (ms_median), and calls following each other over a ring of pool replicas (replica_ring)."""
    import torch
    res = {}
    for name in WORKLOAD_LABEL:
        if name == skip:
            a = cached[1]["attention_only"]
            res[name] = {"unique_kv_bytes": cached[1]["config"]["unique_kv_bytes"], "ms_median": a["ms_median"],
                         "tbps_unique_kv": a["tbps_unique_kv"], "pct_of_8tbps": a["pct_of_8tbps"]}
            continue
        w = load_workload(name)
        b = DeviceBatch(w, dev)
        rsbcm = punch_long_context(rk, b) if name == "long_context" else None
        plan, _ = run_step(rk, b)
        torch.cuda.synchronize()
        kv, _ = algorithmic_bytes(plan, b.w.layout)
        att = attention_only_times(rk, b, plan, 20, flush)
        med = statistics.median(att)
        res[name] = {"unique_kv_bytes": kv, "ms_median": med, "ms_min": min(att),
                     "tbps_unique_kv": kv / (med * 1e-3) / 1e12,
                     "pct_of_8tbps": 100.0 * kv / (med * 1e-3) / 1e12 / NOMINAL_HBM_TBPS,
                     "branch_steps_per_s": b.w.num_branches / (med * 1e-3), "work_items": plan.num_work_items}
        res[name]["replica_ring"] = replica_ring_us(rk, b, plan, kv)
        if name == "diverse_phrasing":
            shared = (b.map_host.numpy() >= 0)
            nonroot = np.arange(shared.size) % 8 != 0
            res[name]["gate_shares_of_non_root_phrasings"] = float(shared[nonroot].mean())
            res[name]["exact_token_cache_would_share"] = float((b.w.phrasing_level == 0)[nonroot].mean())
            res[name]["duplicated_over_unique_kv"] = plan.duplicated_kv_tokens / max(plan.unique_kv_tokens, 1)
        if rsbcm is not None:
            res[name]["rsbcm_eviction_before_this_step"] = rsbcm
        del b
        torch.cuda.empty_cache()
    return res


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
