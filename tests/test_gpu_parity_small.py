"""CUDA path vs the fp64 oracle, element by element, on small and edge-case inputs."""
import dataclasses

import numpy as np
import pytest

import workloads
from helpers import (check_attention, cuda_attention, cuda_gate, oracle_attention, oracle_gate,
                     oracle_tables_from_map)

pytestmark = pytest.mark.gpu


def _parity(w, tables=None):
    ref_out, ref_m = oracle_attention(w, tables)
    out, m, plan = cuda_attention(w, tables)
    return check_attention(out, m, ref_out, ref_m), plan


def test_tiny_as_stated():
    w = workloads.make_tiny()
    err, plan = _parity(w)
    assert plan.unique_kv_tokens == 384 and plan.duplicated_kv_tokens == 1152


def test_tiny_end_to_end_gate_tables_attention():
    import paper_2606_09937_b200 as rk
    w = workloads.make_tiny()
    m_ref, s_ref = oracle_gate(w.gate)
    m, s = cuda_gate(w.gate)
    assert m.tolist() == m_ref.tolist() == workloads.make_tiny_gate_tables()["map"]
    assert np.abs(s - s_ref).max() < 1e-5
    f = w.flat
    t = rk.rksc_tables_from_gate(m, f.num_prefixes, f.shared_off, f.shared_pages, f.shared_ntok,
                                 f.priv_off, f.priv_pages, f.priv_ntok, f.sfx_off, f.sfx_pages, f.sfx_ntok)
    t_ref = oracle_tables_from_map(w, m_ref)
    for k, v in t.as_dict().items():
        assert np.array_equal(v, t_ref[k]), k
    _parity(w, t_ref)


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (28, 4, 128), (32, 8, 128), (4, 4, 128), (16, 1, 64)])
def test_ragged_segments(hq, hkv, d):
    # partial pages, one-token segments, empty segment, empty branch, shared + private mix
    seg_ntok = [37, 5, 16, 1, 0, 100, 17]
    br = [[0, 1], [0, 2], [3], [0, 4, 5], [], [5, 6], [0, 5, 6]]
    w = workloads.make_from_segments("ragged", hq, hkv, d, seg_ntok, br, seed=11)
    _parity(w)


@pytest.mark.parametrize("sharers,G", [(1, 1), (2, 4), (8, 1), (9, 1), (3, 3), (3, 4), (3, 5), (2, 8), (9, 7), (16, 4),
                                       (17, 4), (4, 16), (33, 2), (70, 1)])
def test_row_counts_around_tile_edges(sharers, G):
    # stacked rows = sharers * G: 1, 8, 8 (the last counts of the warp kernel's small-row path), 9, 9, 12, 15,
    # 16 (the first counts of the tcgen05 kernel), 63, 64, 68 (two sharer blocks), 64, 66, 70
    hkv = 2
    w = workloads.make_from_segments("rows", G * hkv, hkv, 128, [200] + [19] * sharers,
                                     [[0, 1 + b] for b in range(sharers)], seed=12 + sharers)
    _parity(w)


@pytest.mark.parametrize("ntok", [1, 3, 17, 64, 130])
@pytest.mark.parametrize("q_gain", [1.0, 6.0])
def test_short_shared_segment_on_the_tensor_core_path(ntok, q_gain):
    # 16 sharers x G = 7 -> 112 stacked rows (the tcgen05 kernel) over a segment of a few tokens, alone:
    # every probability is large, so the rounding of P to bf16 shows in the output if anywhere
    w = workloads.make_from_segments("short_tc", 28, 4, 128, [ntok], [[0]] * 16, seed=40 + ntok, q_gain=q_gain)
    err, plan = _parity(w)
    assert any(plan.item(i)[8] == 1 for i in range(plan.num_work_items))


@pytest.mark.parametrize("ntok", [16, 48, 100, 200])
def test_many_short_items_per_cta_on_the_tensor_core_path(ntok):
    # 300 segments x 4 KV heads = 1200 tensor-core items for 148 CTAs: every CTA runs through several
    # items of one to four slots (its item ring wraps, items owned by one warpgroup only, epilogues
    # with one accumulator empty), each shared by 3 branches x G = 7 -> 21 stacked rows
    nseg = 300
    w = workloads.make_from_segments("many_tc", 28, 4, 128, [ntok] * nseg,
                                     [[s] for s in range(nseg) for _ in range(3)], seed=60 + ntok)
    err, plan = _parity(w)
    assert sum(1 for i in range(plan.num_work_items) if plan.item(i)[8] == 1) >= 1200


def test_long_segment_many_chunks_and_custom_scale():
    w = workloads.make_from_segments("long", 8, 2, 128, [5000, 33, 700], [[0, 1], [0, 2], [0]], seed=13,
                                     sm_scale=0.11)
    err, plan = _parity(w)
    assert plan.num_work_items > 8


@pytest.mark.parametrize("sharers", [1, 24])
def test_very_long_context_against_the_closed_form(sharers):
    """262 144 tokens (16 384 pages, 32 chunks at the 512-page item cap) with identical keys: every score is
    equal, so out = mean of V and every full block holds 16 / T of the mass, whatever the queries - a
    definition the oracle is not needed for at this size.  One branch alone runs the warp path over many
    chunks; 24 sharers x 4 heads run the tensor-core path (96 stacked rows)."""
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    T, Hkv, G, d = 262144, 1, 4, 128
    w = workloads.make_from_segments("maxlen", Hkv * G, Hkv, d, [T], [[0]] * sharers, seed=21)
    key = torch.randn(d, generator=torch.Generator().manual_seed(3)).to(torch.bfloat16)
    pages = torch.from_numpy(np.asarray(w.tables.seg_blocks, dtype=np.int64))
    k_pool = w.k_pool.clone()
    k_pool[pages] = key                                   # the same key in every slot of every listed page
    plan = rk.rksc_plan_create(w.layout, w.tables)
    assert plan.num_work_items >= 32
    out, mass, status = rk.rksc_branch_decode_attention(plan, w.q.to(dev), k_pool.to(dev), w.v_pool.to(dev))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    v_mean = w.v_pool[pages].to(torch.float64).mean(dim=(0, 2)).numpy()          # [Hkv][d]
    got = out.cpu().numpy().astype(np.float64)
    diff = got - v_mean[0][None, None, :]
    assert np.abs(diff).max() <= 2e-4                                            # |mean| ~ 2e-3 per element
    rel = np.linalg.norm(diff, axis=-1) / np.linalg.norm(v_mean[0])
    assert rel.max() <= 1e-2, rel.max()                                          # the relative criterion binds here
    m = rk.split_block_mass(plan, mass)
    for b in range(sharers):
        assert np.abs(m[b].astype(np.float64) - 16.0 / T).max() <= 1e-7
        assert np.abs(m[b].astype(np.float64).sum(axis=1) - 1.0).max() <= 1e-5


def test_tot_small():
    w = workloads.make_tot(root_tokens=300, level_tokens=50)
    _parity(w)


def test_sharp_softmax_large_values():
    # queries scaled x6: near one-hot attention, stresses the running-max rescaling and the abs tolerance
    w = workloads.make_from_segments("sharp", 8, 2, 64, [300, 40], [[0, 1], [0]], seed=14, q_gain=6.0)
    _parity(w)


def test_without_mass_output():
    w = workloads.make_tiny()
    ref_out, _ = oracle_attention(w)
    out, _, _ = cuda_attention(w, want_mass=False)
    check_attention(out, None, ref_out, None)


def test_holes():
    w = workloads.make_long_context(prefix=1500, suffix=70, branches=5, num_q_heads=8, num_kv_heads=2, head_dim=128)
    _, m = oracle_attention(w)
    npg = int(w.tables.seg_block_off[1])
    scores = sum(mb[:, :npg].sum(axis=0) for mb in m)
    h = workloads.punch_holes(w, 0, workloads.lowest_mass_pages(scores, 0.2))
    _parity(h)


def test_gate_edge_cases():
    import torch
    # odd D (scalar path), L not a multiple of anything, several roots, zero-norm layer
    g = workloads.make_gate_inputs([2, 0, 1, 1, 2, 0, 0], 3, 5, 77, [0.0, 0.2, 0.75, 0.1, 2.0, 0.3, float("inf")],
                                   alpha=1.5, tau=0.82, seed=21)
    g.h_branch[3, 2] = 0
    m_ref, s_ref = oracle_gate(g)
    m, s = cuda_gate(g)
    assert np.abs(s - s_ref).max() < 1e-5 and m.tolist() == m_ref.tolist()
    for L, D in ((1, 4), (33, 256), (40, 4096), (64, 100)):
        B = 9
        g = workloads.make_gate_inputs([b % 2 for b in range(B)], 2, L, D,
                                       [0.05 * b for b in range(B)], alpha=0.5, tau=0.9, seed=22 + L)
        m_ref, s_ref = oracle_gate(g)
        m, s = cuda_gate(g)
        assert np.abs(s - s_ref).max() < 1e-5
        clear = np.abs(s_ref - np.float32(0.9)) > 1e-3
        assert np.array_equal(m[clear], m_ref[clear])
