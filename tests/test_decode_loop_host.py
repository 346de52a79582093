"""Host side of the token-by-token decode through the C ABI (no GPU): appended tables vs the oracle."""
import numpy as np
import pytest

import oracle
import workloads


def test_append_matches_oracle_over_many_steps():
    import paper_2606_09937_b200 as rk
    w = workloads.make_from_segments("loop", 28, 4, 128, [37, 21, 16, 0, 300], [[0, 1], [0, 2], [3], [], [0, 4]], seed=5)
    t = w.tables
    ref = {k: getattr(t, k) for k in ("seg_block_off", "seg_blocks", "seg_num_tokens", "br_seg_off", "br_segs")}
    cur = t
    nxt = 1000
    for step in range(40):
        new_pages = np.arange(nxt, nxt + 5, dtype=np.int32)
        nxt += 5
        cur, page, slot = rk.rksc_tables_append_token(cur, new_pages)
        ref, rpage, rslot = oracle.append_token(ref["seg_block_off"], ref["seg_blocks"], ref["seg_num_tokens"],
                                                ref["br_seg_off"], ref["br_segs"], new_pages)
        for k in ref:
            assert getattr(cur, k).tolist() == ref[k].tolist(), (step, k)
        assert page.tolist() == rpage.tolist() and slot.tolist() == rslot.tolist()
    assert cur.seg_num_tokens.tolist() == [37, 61, 56, 40, 340]


def test_append_errors():
    import paper_2606_09937_b200 as rk
    shared_last = workloads.Tables(seg_block_off=np.array([0, 2], np.int32), seg_blocks=np.array([7, 8], np.int32),
                                   seg_num_tokens=np.array([20], np.int32), br_seg_off=np.array([0, 1, 2], np.int32),
                                   br_segs=np.array([0, 0], np.int32))
    with pytest.raises(rk.RkscError) as e:
        rk.rksc_tables_append_token(shared_last, np.array([1, 2], np.int32))
    assert e.value.status == -3
    full = workloads.Tables(seg_block_off=np.array([0, 1], np.int32), seg_blocks=np.array([7], np.int32),
                            seg_num_tokens=np.array([16], np.int32), br_seg_off=np.array([0, 1], np.int32),
                            br_segs=np.array([0], np.int32))
    with pytest.raises(rk.RkscError) as e:
        rk.rksc_tables_append_token(full, None)           # the page is full and no new page is offered
    assert e.value.status == -1
