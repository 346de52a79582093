"""Host side of the RSBCM eviction through the C ABI (no GPU): holed tables vs the oracle."""
import numpy as np
import pytest

import oracle
import workloads


def _same(t, ref):
    o, b, n = ref
    assert t.seg_block_off.tolist() == o.tolist()
    assert t.seg_blocks.tolist() == b.tolist()
    assert t.seg_num_tokens.tolist() == n.tolist()


@pytest.mark.parametrize("make", [workloads.make_tiny, lambda: workloads.make_tot(head_dim=64, num_q_heads=4, num_kv_heads=2,
                                                                                   root_tokens=50, level_tokens=21,
                                                                                   branching=2, depth=2)])
def test_drop_evicted_matches_oracle(make):
    import paper_2606_09937_b200 as rk
    w = make()
    t = w.tables
    n = int(t.seg_block_off[-1])
    rng = np.random.default_rng(11)
    for frac in (0.0, 0.3, 1.0):
        ev = rng.random(n) < frac
        got = rk.rksc_tables_drop_evicted(t, ev)
        _same(got, oracle.apply_eviction(t.seg_block_off, t.seg_blocks, t.seg_num_tokens, ev))
        assert got.br_seg_off.tolist() == t.br_seg_off.tolist() and got.br_segs.tolist() == t.br_segs.tolist()
        # the holed tables are valid input to a plan
        plan = rk.rksc_plan_create(w.layout, got)
        assert plan.num_pages_listed == n - int(ev.sum())


def test_drop_evicted_rejects_bad_tables():
    import paper_2606_09937_b200 as rk
    w = workloads.make_tiny()
    t = w.tables
    bad = workloads.Tables(seg_block_off=t.seg_block_off, seg_blocks=t.seg_blocks,
                           seg_num_tokens=t.seg_num_tokens + 16, br_seg_off=t.br_seg_off, br_segs=t.br_segs)
    with pytest.raises(rk.RkscError) as e:
        rk.rksc_tables_drop_evicted(bad, np.zeros(int(t.seg_block_off[-1]), np.uint8))
    assert e.value.status == -3


def test_workspace_size_rule():
    import paper_2606_09937_b200 as rk
    assert rk.rksc_rsbcm_workspace_bytes(0) == 256
    assert rk.rksc_rsbcm_workspace_bytes(1) == 256
    assert rk.rksc_rsbcm_workspace_bytes(33) == 512
    assert rk.rksc_rsbcm_workspace_bytes(1 << 20) == 8 << 20
