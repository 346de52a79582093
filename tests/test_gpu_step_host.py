"""rksc_decode_step_host: the whole path (gate, map to the host, tables, plan, attention, merge) for
per-step data that lives in host memory, against the oracle run stage by stage.

This is the call the bench's end-to-end figure times.  Map bit-exact, sigma close, outputs and block
masses within the path's tolerances, the mass offsets equal to the plan's; repeated calls (the second
with other queries) check that the library-owned buffers carry nothing over.
"""
import numpy as np
import pytest

import workloads
from helpers import check_attention, oracle_attention, oracle_gate, oracle_tables_from_map

pytestmark = pytest.mark.gpu


def _run(rk, torch, w, q_host, dev_pools):
    g, L = w.gate, w.layout
    B = w.num_branches
    m_host = torch.full((B,), -7, dtype=torch.int32).pin_memory()
    s_host = torch.full((B,), float("nan"), dtype=torch.float32).pin_memory()
    out_host = torch.full((B, L.num_q_heads, L.head_dim), float("nan"), dtype=torch.float32).pin_memory()
    # capacity for the worst case: every branch on a private prefix
    f = w.flat
    worst = int(sum(max(len(f.shared_pages[f.shared_off[g.cand_prefix[b]]:f.shared_off[g.cand_prefix[b] + 1]]),
                        int(f.priv_off[b + 1] - f.priv_off[b])) + int(f.sfx_off[b + 1] - f.sfx_off[b])
                    for b in range(B)))
    mass_host = torch.full((worst * L.num_q_heads,), float("nan"), dtype=torch.float32).pin_memory()
    mass_off = np.zeros(B + 1, dtype=np.int64)
    st = rk.rksc_decode_step_host(L, g.h_branch.pin_memory(), g.h_root.pin_memory(), g.cand_prefix, g.alpha, g.tau,
                                  f, q_host, dev_pools[0], dev_pools[1], m_host, s_host, out_host, mass_host, mass_off)
    assert st == 0
    return m_host.numpy().copy(), s_host.numpy().copy(), out_host.numpy().copy(), mass_host.numpy().copy(), mass_off


@pytest.mark.parametrize("name", ["tiny", "qwen_layer", "diverse_phrasing"])
def test_host_buffer_step_matches_the_oracle_stage_by_stage(name):
    import dataclasses
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    w = workloads.make_config(name)
    pools = (w.k_pool.to(dev), w.v_pool.to(dev))
    m_ref, s_ref = oracle_gate(w.gate)
    t_ref = oracle_tables_from_map(w, m_ref)
    Hq = w.layout.num_q_heads
    sample = None if w.num_branches <= 8 else [0, 2, 5, 7, w.num_branches - 1]
    for call in range(2):
        wq = w if call == 0 else dataclasses.replace(w, q=torch.flip(w.q, dims=[0]).contiguous())
        m, s, out, mass, mass_off = _run(rk, torch, wq, wq.q.pin_memory(), pools)
        assert np.array_equal(m, m_ref)
        assert np.abs(s - s_ref).max() < 1e-5
        ref_out, ref_mass = oracle_attention(wq, t_ref, branches=sample)
        todo = range(w.num_branches) if sample is None else sample
        masses = [None] * w.num_branches
        for b in todo:
            lo, hi = int(mass_off[b]) * Hq, int(mass_off[b + 1]) * Hq
            masses[b] = mass[lo:hi].reshape(Hq, -1)
        nblk = [int(mass_off[b + 1] - mass_off[b]) for b in range(w.num_branches)]
        assert nblk == [int(sum(t_ref["seg_block_off"][sg + 1] - t_ref["seg_block_off"][sg]
                                for sg in t_ref["br_segs"][t_ref["br_seg_off"][b]:t_ref["br_seg_off"][b + 1]]))
                        for b in range(w.num_branches)]
        check_attention(out, masses, ref_out, ref_mass, branches=None if sample is None else sample)
