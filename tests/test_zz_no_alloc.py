"""The allocation-free attention entry point against the regular one.

Some users of the library cannot allocate device memory at call time (a server that gave all
of it to its own pool at start-up, a plug-in barred from the allocating CUDA calls, a latency
path that must not trigger an allocation's device-wide synchronisation).
rksc_branch_decode_attention_static serves them: its partial-result scratch is an array
compiled into the library.  This file checks, through the C ABI, that it returns what the
regular entry point returns - on two calls in a row, because the scratch keeps the previous
call's contents - and that a plan too large for the built-in scratch is refused.  It is named
to be collected last, so that a run that stops at the first failure has already run every
other test.
"""
import numpy as np
import pytest

import workloads


def test_oversized_plan_is_refused_before_any_launch():
    # host-only check: works without a GPU (the size test comes first)
    import paper_2606_09937_b200 as rk
    # many branches x heads -> more partial rows than the 16 MiB scratch holds
    B = 4096
    w = workloads.make_from_segments("big", 16, 1, 128, [16] * B, [[b] for b in range(B)], seed=5)
    plan = rk.rksc_plan_create(w.layout, w.tables)
    assert plan.workspace_bytes > rk.STATIC_WORKSPACE_BYTES
    st = rk.lib().rksc_branch_decode_attention_static(plan._h, None, None, None, None, None, None, None)
    assert st == -4   # RKSC_ERR_WORKSPACE


@pytest.mark.gpu
def test_static_scratch_entry_matches_regular_entry_twice():
    import torch
    import paper_2606_09937_b200 as rk
    from helpers import OUT_ATOL, MASS_ATOL

    dev = torch.device("cuda:0")
    # shared prefix (tensor-core path), a 2-sharer segment and private suffixes (warp paths)
    seg_ntok = [700, 130] + [45] * 6
    br = [[0, 1, 2 + b] if b < 2 else [0, 2 + b] for b in range(6)]
    w = workloads.make_from_segments("noalloc", 28, 4, 128, seg_ntok, br, seed=31)
    plan = rk.rksc_plan_create(w.layout, w.tables)
    assert plan.workspace_bytes <= rk.STATIC_WORKSPACE_BYTES
    q, kp, vp = w.q.to(dev), w.k_pool.to(dev), w.v_pool.to(dev)

    ref_out, ref_mass, status = rk.rksc_branch_decode_attention(plan, q, kp, vp)
    torch.cuda.synchronize()
    assert int(status.item()) == 0

    for call in range(2):
        # the caller owns every buffer; a different query on the second call, so that stale
        # partials left in the shared scratch by the first call would show
        q_call = q if call == 0 else torch.flip(q, dims=[0]).contiguous()
        if call == 1:
            ref_out, ref_mass, status = rk.rksc_branch_decode_attention(plan, q_call, kp, vp)
            torch.cuda.synchronize()
        out = torch.full_like(ref_out, float("nan"))
        mass = torch.full_like(ref_mass, float("nan"))
        st = torch.zeros(1, dtype=torch.int32, device=dev)
        rk.rksc_branch_decode_attention_static(plan, q_call, kp, vp, out, mass, st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        assert float((out - ref_out).abs().max()) <= OUT_ATOL
        assert float((mass - ref_mass).abs().max()) <= MASS_ATOL
        assert bool(torch.isfinite(out).all()) and bool(torch.isfinite(mass).all())
