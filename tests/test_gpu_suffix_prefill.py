"""Suffix prefill on the shared cache (Section 2.2; Appendix "Stepwise Batched Decode", step 1): the
library's virtual-branch tables + its decode attention kernels vs the fp64 oracle."""
import numpy as np
import pytest

import oracle
import workloads
from helpers import check_attention

pytestmark = pytest.mark.gpu


def _run(w, s, seed, sample=None):
    import torch
    import paper_2606_09937_b200 as rk
    t = w.tables
    L = w.layout
    B = t.num_branches
    g = torch.Generator().manual_seed(seed)
    q = torch.randn((B, s, L.num_q_heads, L.head_dim), generator=g, dtype=torch.float32).to(torch.bfloat16)
    vt = rk.rksc_tables_for_suffix_prefill(t, s)
    ref_t = oracle.suffix_prefill_tables(t.seg_block_off, t.seg_blocks, t.seg_num_tokens, t.br_seg_off, t.br_segs, s)
    for k, v in vt.as_dict().items():
        assert np.array_equal(v, ref_t[k]), k                         # bit-exact tables
    plan = rk.rksc_plan_create(L, vt)
    dev = torch.device("cuda:0")
    out, mass, status = rk.rksc_branch_decode_attention(plan, q.reshape(B * s, L.num_q_heads, L.head_dim).to(dev),
                                                        w.k_pool.to(dev), w.v_pool.to(dev))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    masses = rk.split_block_mass(plan, mass)
    branches = range(B) if sample is None else sample
    ref_out, ref_m = oracle.suffix_prefill_attention(
        L.num_q_heads, L.num_kv_heads, L.head_dim, L.sm_scale, t.seg_block_off, t.seg_blocks, t.seg_num_tokens,
        t.br_seg_off, t.br_segs, oracle.to_f32_numpy(q), oracle.to_f32_numpy(w.k_pool), oracle.to_f32_numpy(w.v_pool),
        branches=branches)
    virt = [b * s + i for b in branches for i in range(s)]
    ref_rows = {b * s + i: ref_out[b, i] for b in branches for i in range(s)}
    ref_mass = {}
    for b in branches:
        for i in range(s):
            n = masses[b * s + i].shape[1]
            assert np.all(ref_m[b][i][:, n:] == 0)                    # blocks not listed hold only later tokens
            ref_mass[b * s + i] = ref_m[b][i][:, :n]
    nv = B * s
    check_attention(out.cpu().numpy(), masses, [ref_rows.get(v) for v in range(nv)],
                    [ref_mass.get(v) for v in range(nv)], branches=virt)
    return plan


@pytest.mark.parametrize("hq,hkv,d", [(4, 2, 64), (28, 4, 128), (32, 8, 128)])
@pytest.mark.parametrize("s", [1, 5, 16])
def test_small(hq, hkv, d, s):
    # shared prefix of 37 tokens; own segments of 21, 40 and 16 tokens (16: nothing but the s tokens at s = 16),
    # a branch without a prefix, an empty branch
    w = workloads.make_from_segments("sp", hq, hkv, d, [37, 21, 40, 16, 300, 0],
                                     [[0, 1], [0, 2], [0, 3], [4], [], [0, 4]], seed=70 + s)
    _run(w, s, seed=7)


def test_qwen_shaped_layer_s16():
    # the paper's setting: B branches on one shared prefix, s = 16 suffix tokens (Table of hyperparameters)
    w = workloads.make_qwen_layer(prefix=2048, suffix=16 + 96)
    plan = _run(w, 16, seed=8)
    # the prefix is shared by 4 branches x 16 tokens x G = 7 rows: tensor-core items, and read once per row block
    assert any(plan.item(i)[8] == 1 for i in range(plan.num_work_items))


def test_batched_serving_small_sampled():
    w = workloads.make_batched_serving(problems=3, branches_per=6, prefix_range=(600, 1500), suffix_range=(40, 200))
    from helpers import oracle_gate, oracle_tables_from_map
    d = oracle_tables_from_map(w, oracle_gate(w.gate)[0])
    w.tables = workloads.Tables(**{k: np.asarray(v, np.int32) for k, v in d.items()})
    _run(w, 16, seed=9, sample=[0, 7, 17])
