"""CUDA path vs the oracle on the five configurations at full size, in the launch setup bench.py times.

Small configs are compared element by element; on the large ones the oracle computes a sample of
branches one by one (every sampled branch is compared in full), and properties that hold at any size
(masses sum to 1, finite outputs) are checked for all branches.
"""
import numpy as np
import pytest

import workloads
from helpers import (MASS_SUM_ATOL, check_attention, cuda_attention, cuda_gate, oracle_attention,
                     oracle_gate, oracle_tables_from_map)

pytestmark = pytest.mark.gpu


def _all_branch_properties(out, masses):
    assert np.isfinite(out).all()
    for m in masses:
        if m.size:
            assert np.isfinite(m).all() and (m >= 0).all()
            assert np.abs(m.astype(np.float64).sum(axis=1) - 1.0).max() <= MASS_SUM_ATOL


def _gate_and_tables(w):
    import paper_2606_09937_b200 as rk
    m_ref, s_ref = oracle_gate(w.gate)
    assert np.abs(s_ref - np.float32(w.gate.tau)).min() >= 1e-3       # inputs keep clear of tau
    m, s = cuda_gate(w.gate)
    assert np.array_equal(m, m_ref)                                    # bit-exact map
    assert np.abs(s - s_ref).max() < 1e-5
    f = w.flat
    t = rk.rksc_tables_from_gate(m, f.num_prefixes, f.shared_off, f.shared_pages, f.shared_ntok,
                                 f.priv_off, f.priv_pages, f.priv_ntok, f.sfx_off, f.sfx_pages, f.sfx_ntok)
    t_ref = oracle_tables_from_map(w, m_ref)
    for k, v in t.as_dict().items():
        assert np.array_equal(v, t_ref[k]), k                          # bit-exact tables
    return t_ref


def test_config1_tiny_full():
    w = workloads.make_config("tiny")
    t = _gate_and_tables(w)
    for tables in (w.tables, t):          # as stated (4 sharers) and end to end (3 sharers + private copy)
        ref_out, ref_m = oracle_attention(w, tables)
        out, m, _ = cuda_attention(w, tables)
        check_attention(out, m, ref_out, ref_m)


def test_config2_qwen_layer_full():
    w = workloads.make_config("qwen_layer")
    t = _gate_and_tables(w)
    ref_out, ref_m = oracle_attention(w, t)
    out, m, plan = cuda_attention(w, t)
    check_attention(out, m, ref_out, ref_m)
    assert plan.unique_kv_tokens * w.layout.bytes_per_token == 8 << 20


def test_config3_tot_full():
    w = workloads.make_config("tot")
    out, m, plan = cuda_attention(w)
    _all_branch_properties(out, m)
    assert plan.unique_kv_tokens == 22528 and plan.duplicated_kv_tokens == 114688
    sample = [0, 1, 5, 17, 31, 42, 63]
    ref_out, ref_m = oracle_attention(w, branches=sample)
    check_attention(out, m, ref_out, ref_m, branches=sample)


def test_config4_batched_serving_full():
    w = workloads.make_config("batched_serving")
    t = _gate_and_tables(w)
    m_ref = np.where(w.gate.built_below_tau, -1, w.gate.cand_prefix)
    assert int((m_ref < 0).sum()) == 77
    out, m, plan = cuda_attention(w, t)
    _all_branch_properties(out, m)
    rng = np.random.default_rng(7)
    priv = np.flatnonzero(w.gate.built_below_tau)
    shared = np.flatnonzero(~w.gate.built_below_tau)
    sample = sorted(set(rng.choice(priv, 6, replace=False).tolist() + rng.choice(shared, 10, replace=False).tolist()))
    ref_out, ref_m = oracle_attention(w, t, branches=sample)
    check_attention(out, m, ref_out, ref_m, branches=sample)


def test_config5_long_context_with_holes_full():
    w = workloads.make_config("long_context")
    # eviction choice from the ORACLE's prior-step masses on three sampled branches x all heads,
    # so that both sides get the same holed table and no oracle input comes from the GPU
    prior = [0, 7, 15]
    _, pm = oracle_attention(w, branches=prior)
    npg = int(w.tables.seg_block_off[1])
    scores = sum(pm[b][:, :npg].sum(axis=0) for b in prior)
    ev = workloads.lowest_mass_pages(scores, 0.2)
    assert len(ev) == 409
    h = workloads.punch_holes(w, 0, ev)
    assert int(h.tables.seg_block_off[1]) == 1639
    out, m, plan = cuda_attention(h)
    _all_branch_properties(out, m)
    assert plan.unique_kv_tokens == 1639 * 16 + 16 * 2048
    sample = [0, 9, 15]
    ref_out, ref_m = oracle_attention(h, branches=sample)
    check_attention(out, m, ref_out, ref_m, branches=sample)


def test_config4_through_the_step_pipeline_as_bench_times_it():
    """The launch configuration of the headline loop: config 4 through rksc_pipeline, four steps in
    flight, the same inputs every step.  Every step's map is bit-exact, and the outputs and masses of
    sampled branches of the first and the last step match the oracle."""
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    w = workloads.make_config("batched_serving")
    g, f = w.gate, w.flat
    B, Hq, d = w.num_branches, w.layout.num_q_heads, w.layout.head_dim
    m_ref, s_ref = oracle_gate(g)
    t_ref = oracle_tables_from_map(w, m_ref)
    cap = 0
    for b in range(B):
        r = int(g.cand_prefix[b])
        cap += max(int(f.shared_off[r + 1] - f.shared_off[r]), int(f.priv_off[b + 1] - f.priv_off[b]))
        cap += int(f.sfx_off[b + 1] - f.sfx_off[b])
    cap *= Hq
    depth, n = 4, 6
    pipe = rk.Pipeline(w.layout, B, tuple(g.h_branch.shape[1:]), g.alpha, g.tau, f, depth=depth, mass_capacity=cap,
                       timing=True)
    hb, hr = g.h_branch.to(dev), g.h_root.to(dev)
    cand = torch.from_numpy(g.cand_prefix).to(dev)
    q, kp, vp = w.q.to(dev), w.k_pool.to(dev), w.v_pool.to(dev)
    outs = [torch.full((B, Hq, d), float("nan"), dtype=torch.float32, device=dev) for _ in range(n)]
    masses = [torch.full((cap,), float("nan"), dtype=torch.float32, device=dev) for _ in range(n)]
    torch.cuda.synchronize()
    res = {}
    for i in range(n):
        if i >= depth:
            res[i - depth] = pipe.wait(i - depth)
        pipe.submit(hb, hr, cand, q, kp, vp, outs[i], masses[i])
    for i in range(n - depth, n):
        res[i] = pipe.wait(i)
    pipe.close()
    rng = np.random.default_rng(11)
    priv = np.flatnonzero(g.built_below_tau)
    shared = np.flatnonzero(~g.built_below_tau)
    sample = sorted(set(rng.choice(priv, 4, replace=False).tolist() + rng.choice(shared, 8, replace=False).tolist()))
    ref_out, ref_m = oracle_attention(w, t_ref, branches=sample)
    for i in range(n):
        assert res[i].status == 0 and np.array_equal(res[i].branch_to_prefix, m_ref)
        assert np.abs(res[i].sigma - s_ref).max() < 1e-5
        assert res[i].segment_ms > 0.0
    for i in (0, n - 1):
        flat = masses[i].cpu().numpy()
        ms = [None] * B
        for b in sample:
            lo, hi = int(res[i].mass_off[b]) * Hq, int(res[i].mass_off[b + 1]) * Hq
            ms[b] = flat[lo:hi].reshape(Hq, -1)
        check_attention(outs[i].cpu().numpy(), ms, ref_out, ref_m, branches=sample)
    assert torch.equal(outs[0], outs[n - 1])      # same inputs, same plan, same arithmetic


@pytest.mark.parametrize("name,calls", [("batched_serving", 150), ("tot", 60), ("qwen_layer", 60)])
def test_repeated_calls_are_bitwise_identical_on_a_poisoned_workspace(name, calls):
    """The kernels claim work dynamically, but every item's arithmetic and the merge order are fixed: the
    same call must give the same bits every time, whatever the workspace held before (it is filled with
    NaN bytes between calls, so a partial result that is read before it is written cannot hide).  A
    barrier wait that lets a warp through too early shows up here as a rare difference - so many calls."""
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    w = workloads.make_config(name)
    if w.tables is not None:
        tables = w.tables
    else:
        m_ref, _ = oracle_gate(w.gate)
        tables = oracle_tables_from_map(w, m_ref)
    plan = rk.rksc_plan_create(w.layout, tables)
    q, kp, vp = w.q.to(dev), w.k_pool.to(dev), w.v_pool.to(dev)
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    ref = None
    for i in range(calls):
        ws.fill_(0xFF)
        out, mass, status = rk.rksc_branch_decode_attention(plan, q, kp, vp, workspace=ws)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        if ref is None:
            ref = (out, mass)
            assert bool(torch.isfinite(out).all()) and bool(torch.isfinite(mass).all())
        else:
            assert torch.equal(out, ref[0]), f"call {i}: outputs differ by {float((out - ref[0]).abs().max())}"
            assert torch.equal(mass, ref[1]), f"call {i}: masses differ"


def test_suffix_prefill_calls_are_bitwise_identical_whichever_cta_takes_which_item():
    """Many tensor-core items per CTA, claimed dynamically: the two warpgroups of a CTA split an item's
    slots by the parity of the CTA's running slot count, so an item may find them in either role; the
    item epilogue combines their states symmetrically, and the result has the same bits every time."""
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    w = workloads.make_config("qwen_layer")
    m_ref, _ = oracle_gate(w.gate)
    vt = rk.rksc_tables_for_suffix_prefill(oracle_tables_from_map(w, m_ref), 16)
    plan = rk.rksc_plan_create(w.layout, vt)
    assert plan.num_work_items > 2 * 148          # more items than CTAs: some CTA runs several
    g = torch.Generator().manual_seed(5)
    q = torch.randn((plan.num_branches, w.layout.num_q_heads, w.layout.head_dim), generator=g).to(torch.bfloat16).to(dev)
    kp, vp = w.k_pool.to(dev), w.v_pool.to(dev)
    ws = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    ref = None
    for i in range(60):
        ws.fill_(0xFF)
        out, mass, status = rk.rksc_branch_decode_attention(plan, q, kp, vp, workspace=ws)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        if ref is None:
            ref = (out, mass)
        else:
            assert torch.equal(out, ref[0]) and torch.equal(mass, ref[1]), f"call {i}"


def test_two_plans_on_two_streams_at_once_give_their_single_stream_bits():
    """Distinct plans on distinct streams may run at the same time (the header's promise): their persistent
    kernels then share the SMs, and each call must still give exactly what it gives alone."""
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")

    def prepare(name):
        w = workloads.make_config(name)
        t = w.tables if w.tables is not None else oracle_tables_from_map(w, oracle_gate(w.gate)[0])
        plan = rk.rksc_plan_create(w.layout, t)
        x = dict(plan=plan, q=w.q.to(dev), kp=w.k_pool.to(dev), vp=w.v_pool.to(dev),
                 ws=torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev))
        out, mass, status = rk.rksc_branch_decode_attention(plan, x["q"], x["kp"], x["vp"], workspace=x["ws"])
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        x["ref"] = (out.clone(), mass.clone())
        return x

    pair = [prepare("tot"), prepare("diverse_phrasing")]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for i in range(30):
        res = []
        for x, s in zip(pair, streams):
            with torch.cuda.stream(s):
                x["ws"].fill_(0xFF)
                res.append(rk.rksc_branch_decode_attention(x["plan"], x["q"], x["kp"], x["vp"], workspace=x["ws"],
                                                           stream=s))
        torch.cuda.synchronize()
        for x, (out, mass, status) in zip(pair, res):
            assert int(status.item()) == 0
            assert torch.equal(out, x["ref"][0]) and torch.equal(mass, x["ref"][1]), f"round {i}"


def test_long_prefix_serving_sampled():
    """The larger batch the bench also times (2.4 GB of unique KV: prefixes of 4096-16384 tokens, short
    suffixes): gate map and tables bit-exact, sampled branches against the oracle, properties for all."""
    w = workloads.make_config("long_prefix_serving")
    t = _gate_and_tables(w)
    out, m, plan = cuda_attention(w, t)
    _all_branch_properties(out, m)
    rng = np.random.default_rng(5)
    priv = np.flatnonzero(w.gate.built_below_tau)
    shared = np.flatnonzero(~w.gate.built_below_tau)
    sample = sorted(set(rng.choice(priv, 3, replace=False).tolist() + rng.choice(shared, 5, replace=False).tolist()))
    ref_out, ref_m = oracle_attention(w, t, branches=sample)
    check_attention(out, m, ref_out, ref_m, branches=sample)


def test_late_merge_gives_the_same_bits_and_bad_phase_words_are_refused():
    """RKSC_PHASE_MERGE_LATE only changes how the merge kernel is launched (an ordinary successor instead
    of programmatic serialisation), not what it computes."""
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    w = workloads.make_config("qwen_layer")
    t = oracle_tables_from_map(w, oracle_gate(w.gate)[0])
    plan = rk.rksc_plan_create(w.layout, t)
    q, kp, vp = w.q.to(dev), w.k_pool.to(dev), w.v_pool.to(dev)
    out0, mass0, _ = rk.rksc_branch_decode_attention(plan, q, kp, vp)
    out1, mass1, st = rk.rksc_branch_decode_attention(plan, q, kp, vp, phases=1 | 2 | 4)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and torch.equal(out0, out1) and torch.equal(mass0, mass1)
    for bad in (0, 4, 8, 16 | 1):
        with pytest.raises(rk.RkscError):
            rk.rksc_branch_decode_attention(plan, q, kp, vp, phases=bad)
