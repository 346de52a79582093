"""Host side of the suffix prefill through the C ABI (no GPU): virtual tables vs the oracle."""
import numpy as np
import pytest

import oracle
import workloads


def _same(t, ref):
    for k in ("seg_block_off", "seg_blocks", "seg_num_tokens", "br_seg_off", "br_segs"):
        assert getattr(t, k).tolist() == ref[k].tolist(), k


@pytest.mark.parametrize("s", [1, 3, 16])
def test_tables_match_oracle(s):
    import paper_2606_09937_b200 as rk
    w = workloads.make_from_segments("sp", 28, 4, 128, [37, 21, 40, 16, 300, 0],
                                     [[0, 1], [0, 2], [0, 3], [4], [], [0, 4]], seed=3)
    t = w.tables
    got = rk.rksc_tables_for_suffix_prefill(t, s)
    ref = oracle.suffix_prefill_tables(t.seg_block_off, t.seg_blocks, t.seg_num_tokens, t.br_seg_off, t.br_segs, s)
    _same(got, ref)
    plan = rk.rksc_plan_create(w.layout, got)          # valid input to a plan
    assert plan.num_branches == t.num_branches * s


def test_tables_hand_case_and_errors():
    import paper_2606_09937_b200 as rk
    t = workloads.Tables(seg_block_off=np.array([0, 2, 5], np.int32), seg_blocks=np.array([7, 8, 3, 4, 5], np.int32),
                         seg_num_tokens=np.array([20, 35], np.int32), br_seg_off=np.array([0, 2], np.int32),
                         br_segs=np.array([0, 1], np.int32))
    got = rk.rksc_tables_for_suffix_prefill(t, 4)
    assert got.seg_num_tokens.tolist() == [20, 35, 16, 16, 17, 18, 19]
    assert got.br_segs.tolist() == [0, 2, 3, 0, 2, 4, 0, 2, 5, 0, 2, 6]
    with pytest.raises(rk.RkscError) as e:
        rk.rksc_tables_for_suffix_prefill(t, 36)       # the last segment holds 35 tokens
    assert e.value.status == -3
    with pytest.raises(rk.RkscError) as e:
        rk.rksc_tables_for_suffix_prefill(t, 0)
    assert e.value.status == -1
