"""rksc_pipeline_*: whole steps kept several deep in flight by the library's own streams and threads.

Host tests: the argument checks, and that creation fails loudly without a device (no CPU fallback).
GPU tests: every step that went through the pipeline equals the oracle run stage by stage (gate map
bit-exact, outputs and masses within the path's tolerances) although the steps overlap in time and
differ in queries and in gate inputs (so in tables and plans); the in-flight rules; the refusal of
a mass buffer that is too small; the segment-kernel timing.
"""
import dataclasses

import numpy as np
import pytest

import workloads
from helpers import check_attention, oracle_attention, oracle_gate, oracle_tables_from_map


def test_create_checks_its_arguments_before_touching_the_device():
    import paper_2606_09937_b200 as rk
    w = workloads.make_config("tiny")
    for depth in (1, 9):
        with pytest.raises(rk.RkscError) as e:
            rk.Pipeline(w.layout, w.num_branches, (4, 256), 0.5, 0.9, w.flat, depth=depth)
        assert e.value.status == -1
    with pytest.raises(rk.RkscError) as e:
        rk.Pipeline(w.layout, w.num_branches, (4, 256), 0.5, 0.9, w.flat, depth=4, mass_capacity=-5)
    assert e.value.status == -1


def test_create_fails_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    import paper_2606_09937_b200 as rk
    w = workloads.make_config("tiny")
    with pytest.raises(rk.RkscError) as e:
        rk.Pipeline(w.layout, w.num_branches, (4, 256), 0.5, 0.9, w.flat, depth=4)
    assert e.value.status == -5     # RKSC_ERR_CUDA: nothing is computed on the host instead


def _mass_capacity(w):
    f, g = w.flat, w.gate
    pages = 0
    for b in range(w.num_branches):
        r = int(g.cand_prefix[b])
        pages += max(int(f.shared_off[r + 1] - f.shared_off[r]), int(f.priv_off[b + 1] - f.priv_off[b]))
        pages += int(f.sfx_off[b + 1] - f.sfx_off[b])
    return pages * w.layout.num_q_heads


def _variants(w, n):
    """n steps' inputs: queries rotated along the branch axis; every other step one more branch is
    drawn independently of its root (it loses its share, so tables and plan differ between steps)."""
    import torch
    steps = []
    for i in range(n):
        q = torch.roll(w.q, shifts=i, dims=0).contiguous()
        hb = w.gate.h_branch
        if i % 2 == 1 and w.num_branches > 2:
            hb = hb.clone()
            g = torch.Generator().manual_seed(1000 + i)
            hb[1] = torch.randn(hb[1].shape, generator=g)      # sigma about 0: far below tau
        gate = dataclasses.replace(w.gate, h_branch=hb)
        steps.append(dataclasses.replace(w, q=q, gate=gate))
    return steps


@pytest.mark.gpu
@pytest.mark.parametrize("name,depth", [("tiny", 4), ("qwen_layer", 3), ("diverse_phrasing", 4), ("tiny", 2)])
def test_steps_through_the_pipeline_match_the_oracle(name, depth):
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    w = workloads.make_config(name)
    n = 7
    steps = _variants(w, n)
    L, D = w.gate.h_branch.shape[1:]
    cap = _mass_capacity(w)
    pipe = rk.Pipeline(w.layout, w.num_branches, (L, D), w.gate.alpha, w.gate.tau, w.flat, depth=depth,
                       mass_capacity=cap)
    kp, vp = w.k_pool.to(dev), w.v_pool.to(dev)
    hr = w.gate.h_root.to(dev)
    cand = torch.from_numpy(w.gate.cand_prefix).to(dev)
    Hq, d = w.layout.num_q_heads, w.layout.head_dim
    outs = [torch.full((w.num_branches, Hq, d), float("nan"), dtype=torch.float32, device=dev) for _ in range(n)]
    masses = [torch.full((cap,), float("nan"), dtype=torch.float32, device=dev) for _ in range(n)]
    hbs = [s.gate.h_branch.to(dev) for s in steps]
    qs = [s.q.to(dev) for s in steps]
    torch.cuda.synchronize()
    results = {}
    for i in range(n):
        if i >= depth:
            results[i - depth] = pipe.wait(i - depth)
        t = pipe.submit(hbs[i], hr, cand, qs[i], kp, vp, outs[i], masses[i])
        assert t == i
    for i in range(max(0, n - depth), n):
        results[i] = pipe.wait(i)
    pipe.close()

    sample = None if w.num_branches <= 8 else [0, 1, 2, 5, w.num_branches - 1]
    for i, s in enumerate(steps):
        r = results[i]
        m_ref, s_ref = oracle_gate(s.gate)
        assert np.abs(s_ref - np.float32(s.gate.tau)).min() >= 1e-3
        assert np.array_equal(r.branch_to_prefix, m_ref), i
        assert np.abs(r.sigma - s_ref).max() < 1e-5
        t_ref = oracle_tables_from_map(s, m_ref)
        ref_out, ref_mass = oracle_attention(s, t_ref, branches=sample)
        flat = masses[i].cpu().numpy()
        ms = [None] * w.num_branches
        for b in (range(w.num_branches) if sample is None else sample):
            lo, hi = int(r.mass_off[b]) * Hq, int(r.mass_off[b + 1]) * Hq
            ms[b] = flat[lo:hi].reshape(Hq, -1)
        check_attention(outs[i].cpu().numpy(), ms, ref_out, ref_mass, branches=sample)
    if w.num_branches > 2:
        assert not np.array_equal(results[0].branch_to_prefix, results[1].branch_to_prefix)   # the plans did differ


@pytest.mark.gpu
def test_in_flight_rules_small_mass_buffer_and_timing():
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    w = workloads.make_config("tiny")
    L, D = w.gate.h_branch.shape[1:]
    cap = _mass_capacity(w)
    hb, hr = w.gate.h_branch.to(dev), w.gate.h_root.to(dev)
    cand = torch.from_numpy(w.gate.cand_prefix).to(dev)
    q, kp, vp = w.q.to(dev), w.k_pool.to(dev), w.v_pool.to(dev)
    out = torch.empty((w.num_branches, w.layout.num_q_heads, w.layout.head_dim), dtype=torch.float32, device=dev)
    mass = torch.empty(cap, dtype=torch.float32, device=dev)

    pipe = rk.Pipeline(w.layout, w.num_branches, (L, D), w.gate.alpha, w.gate.tau, w.flat, depth=2, mass_capacity=cap,
                       timing=True)
    assert pipe.submit(hb, hr, cand, q, kp, vp, out, mass) == 0
    assert pipe.submit(hb, hr, cand, q, kp, vp, out, mass) == 1
    with pytest.raises(rk.RkscError):               # two in flight, none waited for
        pipe.submit(hb, hr, cand, q, kp, vp, out, mass)
    assert pipe.wait(1, check=False).status == -1   # out of order
    r0 = pipe.wait(0)
    assert r0.status == 0 and r0.segment_ms > 0.0 and r0.num_kernel_launches >= 2
    assert pipe.wait(0, check=False).status == -1   # twice
    assert pipe.submit(hb, hr, cand, q, kp, vp, out, mass) == 2
    assert pipe.wait(1).status == 0 and pipe.wait(2).status == 0
    pipe.close()

    # timing = 2: events around the segment kernels of every second step only
    every2 = rk.Pipeline(w.layout, w.num_branches, (L, D), w.gate.alpha, w.gate.tau, w.flat, depth=4, mass_capacity=cap,
                         timing=2)
    for i in range(4):
        every2.submit(hb, hr, cand, q, kp, vp, out, mass)
    ms = [every2.wait(i).segment_ms for i in range(4)]
    every2.close()
    assert ms[0] > 0.0 and ms[2] > 0.0 and ms[1] == 0.0 and ms[3] == 0.0

    small = rk.Pipeline(w.layout, w.num_branches, (L, D), w.gate.alpha, w.gate.tau, w.flat, depth=3, mass_capacity=8)
    out.fill_(7.0)
    t = small.submit(hb, hr, cand, q, kp, vp, out, mass)
    r = small.wait(t, check=False)
    assert r.status == -4                            # RKSC_ERR_WORKSPACE, and the attention did not run
    torch.cuda.synchronize()
    assert float(out.min()) == 7.0 and float(out.max()) == 7.0
    m_ref, _ = oracle_gate(w.gate)
    assert np.array_equal(r.branch_to_prefix, m_ref)  # the gate's result is still handed back
    # without a mass buffer the same pipeline runs the step
    t = small.submit(hb, hr, cand, q, kp, vp, out, None)
    assert small.wait(t).status == 0
    # destroying a pipeline with steps in flight finishes them first
    out.fill_(float("nan"))
    torch.cuda.synchronize()
    small.submit(hb, hr, cand, q, kp, vp, out, None)
    small.submit(hb, hr, cand, q, kp, vp, out, None)
    small.close()
    assert bool(torch.isfinite(out).all())


@pytest.mark.gpu
def test_many_steps_at_full_depth_reuse_their_slots_correctly():
    """Forty steps eight deep: every slot is reused five times, gates of later steps run beside the
    attention of earlier ones, and each step's outputs still belong to its own inputs."""
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    w = workloads.make_config("tiny")
    depth, n = 8, 40
    variants = _variants(w, 4)                    # four distinct (query, gate input) pairs, cycled
    refs = []
    for s in variants:
        m_ref, _ = oracle_gate(s.gate)
        refs.append((m_ref,) + tuple(oracle_attention(s, oracle_tables_from_map(s, m_ref))))
    L, D = w.gate.h_branch.shape[1:]
    cap = _mass_capacity(w)
    pipe = rk.Pipeline(w.layout, w.num_branches, (L, D), w.gate.alpha, w.gate.tau, w.flat, depth=depth,
                       mass_capacity=cap)
    kp, vp = w.k_pool.to(dev), w.v_pool.to(dev)
    hr = w.gate.h_root.to(dev)
    cand = torch.from_numpy(w.gate.cand_prefix).to(dev)
    hbs = [s.gate.h_branch.to(dev) for s in variants]
    qs = [s.q.to(dev) for s in variants]
    Hq, d = w.layout.num_q_heads, w.layout.head_dim
    outs = [torch.empty((w.num_branches, Hq, d), dtype=torch.float32, device=dev) for _ in range(depth)]
    masses = [torch.empty(cap, dtype=torch.float32, device=dev) for _ in range(depth)]

    def check(t, r):
        m_ref, ref_out, ref_mass = refs[t % 4]
        assert np.array_equal(r.branch_to_prefix, m_ref), t
        flat = masses[t % depth].cpu().numpy()
        ms = [flat[int(r.mass_off[b]) * Hq:int(r.mass_off[b + 1]) * Hq].reshape(Hq, -1) for b in range(w.num_branches)]
        check_attention(outs[t % depth].cpu().numpy(), ms, ref_out, ref_mass)

    for t in range(n):
        if t >= depth:
            check(t - depth, pipe.wait(t - depth))          # before the slot's buffers are reused
        outs[t % depth].fill_(float("nan"))
        masses[t % depth].fill_(float("nan"))
        assert pipe.submit(hbs[t % 4], hr, cand, qs[t % 4], kp, vp, outs[t % depth], masses[t % depth],
                           after_stream=torch.cuda.current_stream()) == t
    for t in range(n - depth, n):
        check(t, pipe.wait(t))
    pipe.close()
