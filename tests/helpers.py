"""Shared helpers for the tests (input conversion, tolerances)."""
import os

import numpy as np

import oracle

# Tolerances of the target statement: attention outputs within max-abs 2e-3 and
# relative (row 2-norm) 1e-2 of the fp64 oracle; block masses within 1e-4 abs;
# masses of one (branch, head) sum to 1 within 1e-5.
OUT_ATOL = 2e-3
OUT_RTOL = 1e-2
MASS_ATOL = 1e-4
MASS_SUM_ATOL = 1e-5


def golden_facts():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_facts.txt")
    facts = {}
    with open(path) as f:
        for line in f:
            line = line.split("#", 1)[0].strip()
            if not line:
                continue
            parts = line.split()
            vals = [float(v) for v in parts[1:]]
            facts[parts[0]] = vals[0] if len(vals) == 1 else vals
    return facts


def oracle_attention(w, tables=None, branches=None):
    """Run the oracle on a workload; tables default to the workload's given tables."""
    t = tables if tables is not None else w.tables
    get = (lambda k: t[k]) if isinstance(t, dict) else (lambda k: getattr(t, k))
    L = w.layout
    return oracle.branch_decode_attention(
        L.num_q_heads, L.num_kv_heads, L.head_dim, L.sm_scale,
        get("seg_block_off"), get("seg_blocks"), get("seg_num_tokens"),
        get("br_seg_off"), get("br_segs"),
        oracle.to_f32_numpy(w.q), oracle.to_f32_numpy(w.k_pool), oracle.to_f32_numpy(w.v_pool),
        branches=branches)


def oracle_gate(g):
    return oracle.asks_gate(g.h_branch.numpy(), g.h_root.numpy(), g.cand_prefix, g.alpha, g.tau)


def oracle_tables_from_map(w, branch_to_prefix):
    f = w.flat
    return oracle.tables_from_gate(branch_to_prefix, f.num_prefixes,
                                   f.shared_off, f.shared_pages, f.shared_ntok,
                                   f.priv_off, f.priv_pages, f.priv_ntok,
                                   f.sfx_off, f.sfx_pages, f.sfx_ntok)


def check_attention(out, masses, ref_out, ref_masses, branches=None):
    """Assert the target tolerances; returns the error figures."""
    out = np.asarray(out, dtype=np.float64)
    B = out.shape[0]
    todo = range(B) if branches is None else branches
    max_abs = 0.0
    max_rel = 0.0
    max_mass = 0.0
    max_sum = 0.0
    for b in todo:
        d = out[b] - ref_out[b]
        max_abs = max(max_abs, float(np.abs(d).max()))
        nr = np.linalg.norm(ref_out[b], axis=-1)
        nd = np.linalg.norm(d, axis=-1)
        ok = nr > 0
        if ok.any():
            max_rel = max(max_rel, float((nd[ok] / nr[ok]).max()))
        if masses is not None and ref_masses[b] is not None and ref_masses[b].size:
            m = np.asarray(masses[b], dtype=np.float64)
            assert m.shape == ref_masses[b].shape
            max_mass = max(max_mass, float(np.abs(m - ref_masses[b]).max()))
            max_sum = max(max_sum, float(np.abs(m.sum(axis=1) - 1.0).max()))
    assert max_abs <= OUT_ATOL, f"out max-abs {max_abs}"
    assert max_rel <= OUT_RTOL, f"out relative {max_rel}"
    if masses is not None:
        assert max_mass <= MASS_ATOL, f"mass max-abs {max_mass}"
        assert max_sum <= MASS_SUM_ATOL, f"mass sum {max_sum}"
    return {"max_abs": max_abs, "max_rel": max_rel, "max_mass": max_mass, "max_mass_sum": max_sum}


# ---------------------------------------------------------------------------------------
# CUDA path (through the C ABI binding)
# ---------------------------------------------------------------------------------------

def cuda_attention(w, tables=None, want_mass=True, pools=None):
    """Run the library on a workload; returns (out numpy, masses list, plan)."""
    import torch
    import paper_2606_09937_b200 as rk
    t = tables if tables is not None else w.tables
    plan = rk.rksc_plan_create(w.layout, t)
    dev = torch.device("cuda:0")
    if pools is None:
        pools = (w.k_pool.to(dev), w.v_pool.to(dev))
    q = w.q.to(dev)
    out, mass, status = rk.rksc_branch_decode_attention(plan, q, pools[0], pools[1], want_mass=want_mass)
    torch.cuda.synchronize()
    assert int(status.item()) == 0, f"device status {int(status.item())}"
    masses = rk.split_block_mass(plan, mass) if want_mass else None
    return out.cpu().numpy(), masses, plan


def cuda_gate(g):
    import torch
    import paper_2606_09937_b200 as rk
    dev = torch.device("cuda:0")
    m, s = rk.rksc_asks_gate(g.h_branch.to(dev), g.h_root.to(dev),
                             torch.from_numpy(g.cand_prefix).to(dev), g.alpha, g.tau)
    torch.cuda.synchronize()
    return m.cpu().numpy(), s.cpu().numpy()
