"""Pins for the decode-loop oracle (Appendix "Stepwise Batched Decode", step 2)."""
import numpy as np
import pytest

import oracle
import workloads


def test_append_hand_case():
    # segment 0: shared prefix (20 tokens, pages 7, 8); segment 1: 16 tokens in page 3 (full); segment 2: 5 tokens in page 4
    off, blocks, ntok = [0, 2, 3, 4], [7, 8, 3, 4], [20, 16, 5]
    br_off, br_segs = [0, 2, 4, 4], [0, 1, 0, 2]
    t, page, slot = oracle.append_token(off, blocks, ntok, br_off, br_segs, [11, 12, 13])
    assert t["seg_block_off"].tolist() == [0, 2, 4, 5] and t["seg_blocks"].tolist() == [7, 8, 3, 11, 4]
    assert t["seg_num_tokens"].tolist() == [20, 17, 6]
    assert page.tolist() == [11, 4, -1] and slot.tolist() == [0, 5, -1]
    # a shared last segment cannot grow
    with pytest.raises(ValueError):
        oracle.append_token([0, 2], [7, 8], [20], [0, 1, 2], [0, 0], [1, 2])


def test_sixteen_appends_fill_exactly_one_page_and_attention_sees_the_new_tokens():
    w = workloads.make_from_segments("loop", 4, 2, 64, [37, 21, 16, 0], [[0, 1], [0, 2], [3]], seed=5)
    t = {k: getattr(w.tables, k) for k in ("seg_block_off", "seg_blocks", "seg_num_tokens", "br_seg_off", "br_segs")}
    k = oracle.to_f32_numpy(w.k_pool).copy()
    v = oracle.to_f32_numpy(w.v_pool).copy()
    extra = 8
    k = np.concatenate([k, np.zeros((extra,) + k.shape[1:], k.dtype)])
    v = np.concatenate([v, np.zeros((extra,) + v.shape[1:], v.dtype)])
    free = list(range(k.shape[0] - extra, k.shape[0]))
    rng = np.random.default_rng(0)
    pages_before = int(t["seg_block_off"][-1])
    for step in range(16):
        new_pages = [free[(3 * step + b) % extra] for b in range(3)]
        t, page, slot = oracle.append_token(t["seg_block_off"], t["seg_blocks"], t["seg_num_tokens"], t["br_seg_off"],
                                            t["br_segs"], new_pages)
        oracle.write_token(k, v, page, slot, rng.standard_normal((3, 2, 64)), rng.standard_normal((3, 2, 64)))
    # every branch gained 16 tokens = exactly one page each, whatever the fill of its last page was
    assert int(t["seg_block_off"][-1]) == pages_before + 3
    assert t["seg_num_tokens"].tolist() == [37, 37, 32, 16]
    # a query aligned with the last appended key of branch 2 puts nearly all its mass on the last block
    L = w.layout
    s3 = 3
    last_page = int(t["seg_blocks"][t["seg_block_off"][s3 + 1] - 1])
    q = np.zeros((3, 4, 64))
    q[2, :, :] = 40.0 * k[last_page, 0, 15, :] / np.linalg.norm(k[last_page, 0, 15, :])
    out, masses = oracle.branch_decode_attention(L.num_q_heads, L.num_kv_heads, L.head_dim, L.sm_scale, t["seg_block_off"],
                                                 t["seg_blocks"], t["seg_num_tokens"], t["br_seg_off"], t["br_segs"], q, k, v)
    assert masses[2][0, -1] > 0.99
