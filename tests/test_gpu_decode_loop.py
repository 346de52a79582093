"""Token-by-token decode on the paged cache (Appendix "Stepwise Batched Decode", step 2): appended tables and
pools bit-exact against the oracle's, the attention of every step within the path's tolerances."""
import numpy as np
import pytest

import oracle
import workloads
from helpers import check_attention

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("hq,hkv,d", [(8, 2, 64), (28, 4, 128)])
def test_decode_loop(hq, hkv, d):
    import torch
    import paper_2606_09937_b200 as rk
    steps, extra = 20, 16
    w = workloads.make_from_segments("loop", hq, hkv, d, [200, 21, 16, 0, 70, 5], [[0, 1], [0, 2], [0, 3], [4], [], [0, 5]],
                                     seed=9)
    L = w.layout
    B = w.tables.num_branches
    dev = torch.device("cuda:0")
    nblk = w.k_pool.shape[0]
    grow = lambda p: torch.cat([p, torch.zeros((extra,) + tuple(p.shape[1:]), dtype=p.dtype)])
    k_dev, v_dev = grow(w.k_pool).to(dev), grow(w.v_pool).to(dev)
    k_ref = oracle.to_f32_numpy(grow(w.k_pool)).copy()
    v_ref = oracle.to_f32_numpy(grow(w.v_pool)).copy()
    import dataclasses
    lay = dataclasses.replace(L, num_pool_blocks=nblk + extra)
    t = w.tables
    ref = {k: getattr(t, k) for k in ("seg_block_off", "seg_blocks", "seg_num_tokens", "br_seg_off", "br_segs")}
    cur = t
    free = nblk
    gen = torch.Generator().manual_seed(3)
    for step in range(steps):
        new_pages = np.full(B, -1, np.int32)
        # a page for every branch whose last page is full (the allocator's job; here: the next free ones)
        probe, _, _ = oracle.append_token(ref["seg_block_off"], ref["seg_blocks"], ref["seg_num_tokens"], ref["br_seg_off"],
                                          ref["br_segs"], np.arange(10**6, 10**6 + B))
        for b in np.flatnonzero(np.isin(np.arange(10**6, 10**6 + B), probe["seg_blocks"])):
            new_pages[b] = free
            free += 1
        assert free <= nblk + extra
        k_new = torch.randn((B, hkv, d), generator=gen).to(torch.bfloat16)
        v_new = torch.randn((B, hkv, d), generator=gen).to(torch.bfloat16)
        q = torch.randn((B, hq, d), generator=gen).to(torch.bfloat16)
        cur, page, slot = rk.rksc_tables_append_token(cur, new_pages)
        rk.rksc_kv_append(lay, k_dev, v_dev, k_new.to(dev), v_new.to(dev), torch.from_numpy(page).to(dev),
                          torch.from_numpy(slot).to(dev))
        ref, rpage, rslot = oracle.append_token(ref["seg_block_off"], ref["seg_blocks"], ref["seg_num_tokens"],
                                                ref["br_seg_off"], ref["br_segs"], new_pages)
        oracle.write_token(k_ref, v_ref, rpage, rslot, oracle.to_f32_numpy(k_new), oracle.to_f32_numpy(v_new))
        assert page.tolist() == rpage.tolist() and slot.tolist() == rslot.tolist()
        for key in ref:
            assert getattr(cur, key).tolist() == ref[key].tolist(), (step, key)
        if step % 4 == 3 or step == steps - 1:
            plan = rk.rksc_plan_create(lay, cur)
            out, mass, status = rk.rksc_branch_decode_attention(plan, q.to(dev), k_dev, v_dev)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
            ref_out, ref_m = oracle.branch_decode_attention(hq, hkv, d, L.sm_scale, ref["seg_block_off"], ref["seg_blocks"],
                                                            ref["seg_num_tokens"], ref["br_seg_off"], ref["br_segs"],
                                                            oracle.to_f32_numpy(q), k_ref, v_ref)
            check_attention(out.cpu().numpy(), rk.split_block_mass(plan, mass), ref_out, ref_m)
    # the pools, bit for bit (bf16 copies are exact)
    assert np.array_equal(oracle.to_f32_numpy(k_dev.cpu()), k_ref) and np.array_equal(oracle.to_f32_numpy(v_dev.cpu()), v_ref)
