"""The diverse-phrasing regime (Section "ASKS Novelty Over vLLM Prefix Caching") as a workload.

Every problem is posed through eight phrasings at four divergence levels; an exact-token prefix cache
can share only the identical ones, the similarity gate also takes the minor rewordings.  The CPU tests
pin the generator's recipe to the figures the paper states (templates, levels, problems, prefix length,
and the share of extra reuse) through the oracle's gate; the GPU tests run the gate, the tables and the
attention of this workload against the oracle like the five main configurations.
"""
import numpy as np
import pytest

import workloads
from helpers import golden_facts, oracle_gate, oracle_tables_from_map


def _nonroot(w):
    templates = int(golden_facts()["phrasing_templates"])
    return np.arange(w.num_branches) % templates != 0


def test_recipe_matches_the_figures_the_paper_states():
    f = golden_facts()
    w = workloads.make_config("diverse_phrasing")
    assert w.num_branches == int(f["phrasing_problems"]) * int(f["phrasing_templates"])
    assert len(set(w.phrasing_level.tolist())) == int(f["phrasing_levels"])
    assert (w.flat.shared_ntok == int(f["phrasing_prefix_tokens"])).all()
    assert w.gate.alpha == f["alpha_default"] and w.gate.tau == f["tau_default"]


def test_oracle_gate_shares_the_two_closer_levels_and_reproduces_the_extra_reuse():
    f = golden_facts()
    w = workloads.make_config("diverse_phrasing")
    m, sigma = oracle_gate(w.gate)
    assert np.abs(sigma - np.float32(w.gate.tau)).min() >= 1e-3
    shares = m >= 0
    assert np.array_equal(shares, w.phrasing_level <= 1)
    assert np.array_equal(m[shares], w.gate.cand_prefix[shares])
    # identical phrasings: sigma = 1 (Section 2.2), and they are all an exact-token cache can share
    assert np.allclose(sigma[w.phrasing_level == 0], f["identical_prefix_sigma"], atol=1e-12)
    nr = _nonroot(w)
    exact = (w.phrasing_level == 0)[nr].mean()
    extra = (shares & (w.phrasing_level > 0))[nr].mean()
    assert round(100.0 * extra, 1) == f["phrasing_extra_reuse_percent"]
    assert exact + extra == shares[nr].mean()


def test_tables_from_the_map_read_each_shared_prefix_once():
    w = workloads.make_config("diverse_phrasing")
    m, _ = oracle_gate(w.gate)
    t = oracle_tables_from_map(w, m)
    tab = workloads.Tables(**{k: np.asarray(v) for k, v in t.items()})
    P = w.flat.num_prefixes
    # segments: 15 shared prefixes (four sharers each), 60 private copies, 120 suffixes
    assert tab.num_segments == P + int((m < 0).sum()) + w.num_branches
    uniq = workloads.unique_kv_bytes(w.layout, tab)
    dup = workloads.duplicated_kv_bytes(w.layout, tab)
    prefix_bytes = 512 * w.layout.bytes_per_token
    assert dup - uniq == 3 * P * prefix_bytes      # three of the four sharers ride on the first one's pages


@pytest.mark.gpu
def test_gpu_gate_tables_and_attention_on_the_diverse_phrasing_workload():
    import paper_2606_09937_b200 as rk
    from helpers import check_attention, cuda_attention, cuda_gate, oracle_attention, MASS_SUM_ATOL

    w = workloads.make_config("diverse_phrasing")
    m_ref, s_ref = oracle_gate(w.gate)
    m, s = cuda_gate(w.gate)
    assert np.array_equal(m, m_ref)
    assert np.abs(s - s_ref).max() < 1e-5
    f = w.flat
    t = rk.rksc_tables_from_gate(m, f.num_prefixes, f.shared_off, f.shared_pages, f.shared_ntok,
                                 f.priv_off, f.priv_pages, f.priv_ntok, f.sfx_off, f.sfx_pages, f.sfx_ntok)
    t_ref = oracle_tables_from_map(w, m_ref)
    for k, v in t.as_dict().items():
        assert np.array_equal(v, t_ref[k]), k
    out, masses, plan = cuda_attention(w, t_ref)
    assert np.isfinite(out).all()
    for mm in masses:
        assert np.abs(mm.astype(np.float64).sum(axis=1) - 1.0).max() <= MASS_SUM_ATOL
    sample = [0, 1, 3, 4, 7, 58, 119]      # every level, first and last problem
    ref_out, ref_m = oracle_attention(w, t_ref, branches=sample)
    check_attention(out, masses, ref_out, ref_m, branches=sample)
