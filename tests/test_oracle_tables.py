"""Pins for the table oracle and the workload generators (integer work, exact)."""
import numpy as np

import oracle
import workloads
from helpers import golden_facts, oracle_tables_from_map


def test_toy_two_problems_hand_written():
    # 2 prefixes, 4 branches; branch 1 fails the gate, nobody shares prefix 1 except branch 3
    shared = dict(shared_off=[0, 2, 5], shared_pages=[10, 11, 20, 21, 22], shared_ntok=[32, 40])
    priv = dict(priv_off=[0, 0, 2, 2, 2], priv_pages=[30, 31], priv_ntok=[0, 20, 0, 0])
    sfx = dict(sfx_off=[0, 1, 2, 3, 5], sfx_pages=[40, 41, 42, 43, 44], sfx_ntok=[3, 16, 1, 17])
    t = oracle.tables_from_gate([0, -1, 0, 1], 2, **shared, **priv, **sfx)
    # segments: shared 0, shared 1, private(1), suffix 0..3
    assert t["seg_block_off"].tolist() == [0, 2, 5, 7, 8, 9, 10, 12]
    assert t["seg_blocks"].tolist() == [10, 11, 20, 21, 22, 30, 31, 40, 41, 42, 43, 44]
    assert t["seg_num_tokens"].tolist() == [32, 40, 20, 3, 16, 1, 17]
    assert t["br_seg_off"].tolist() == [0, 2, 4, 6, 8]
    assert t["br_segs"].tolist() == [0, 3, 2, 4, 0, 5, 1, 6]
    sh = oracle.segment_sharers(t["br_seg_off"], t["br_segs"], 7)
    assert sh == [[0, 2], [3], [1], [0], [1], [2], [3]]
    n = oracle.logical_block_counts(t["seg_block_off"], t["br_seg_off"], t["br_segs"])
    assert n.tolist() == [3, 3, 3, 5]
    assert oracle.mass_offsets(t["seg_block_off"], t["br_seg_off"], t["br_segs"]).tolist() == [0, 3, 6, 9, 14]
    # a prefix nobody shares gets no segment
    t2 = oracle.tables_from_gate([0, -1, 0, -1], 2, **shared, **priv, **sfx)
    assert t2["seg_num_tokens"].tolist() == [32, 20, 0, 3, 16, 1, 17]
    assert t2["br_segs"].tolist() == [0, 3, 1, 4, 0, 5, 2, 6]


def test_tiny_gate_tables_hand_written():
    w = workloads.make_tiny()
    exp = workloads.make_tiny_gate_tables()
    t = oracle_tables_from_map(w, exp["map"])
    assert t["seg_num_tokens"].tolist() == exp["seg_num_tokens"]
    assert [t["br_segs"][2 * b:2 * b + 2].tolist() for b in range(4)] == exp["br_segs"]
    f = w.flat
    assert t["seg_blocks"][:16].tolist() == f.shared_pages.tolist()
    assert t["seg_blocks"][16:32].tolist() == f.priv_pages.tolist()
    # as-stated tables: all four branches on the shared prefix
    sh = oracle.segment_sharers(w.tables.br_seg_off, w.tables.br_segs, w.tables.num_segments)
    assert sh[0] == [0, 1, 2, 3]


def test_tot_tree_shape():
    facts = golden_facts()
    w = workloads.make_tot(head_dim=64, num_q_heads=2, num_kv_heads=1, root_tokens=32, level_tokens=16)
    t = w.tables
    br, depth = int(facts["tot_branching"]), int(facts["tot_depth"])
    assert t.num_segments == sum(br ** k for k in range(depth + 1)) == 85
    assert t.num_branches == br ** depth == 64
    sh = oracle.segment_sharers(t.br_seg_off, t.br_segs, t.num_segments)
    assert [len(s) for s in sh] == [64] + [16] * 4 + [4] * 16 + [1] * 64
    assert sh[1] == list(range(16)) and sh[5] == [0, 1, 2, 3]
    # two leaves that diverge at depth 2 (same depth-1 and depth-2... i.e. last level differs)
    a = t.br_segs[t.br_seg_off[0]:t.br_seg_off[1]]
    b = t.br_segs[t.br_seg_off[1]:t.br_seg_off[2]]
    shared_levels = sum(int(x == y) for x, y in zip(a[1:], b[1:]))
    assert shared_levels == 2
    assert int(100 * shared_levels / depth) == int(facts["tot_shared_percent_diverging_at_depth2"])


def test_pool_pages_unique_and_in_range():
    for w in (workloads.make_tiny(), workloads.make_tot(head_dim=64, num_q_heads=2, num_kv_heads=1,
                                                        root_tokens=40, level_tokens=24)):
        t = w.tables
        assert len(np.unique(t.seg_blocks)) == len(t.seg_blocks)
        assert t.seg_blocks.min() >= 0 and t.seg_blocks.max() < w.layout.num_pool_blocks
        npages = np.diff(t.seg_block_off)
        assert np.all(npages == (t.seg_num_tokens + 15) // 16)


def test_batched_serving_structure_small():
    w = workloads.make_batched_serving(problems=4, branches_per=8, prefix_range=(20, 70),
                                       suffix_range=(5, 40), L=4, D=512, head_dim=64,
                                       num_q_heads=4, num_kv_heads=2)
    f = w.flat
    assert int(w.gate.built_below_tau.sum()) == round(0.3 * 32)
    for b in range(32):
        has_priv = f.priv_off[b + 1] > f.priv_off[b]
        assert has_priv == bool(w.gate.built_below_tau[b])
        if has_priv:
            assert f.priv_ntok[b] == f.shared_ntok[b // 8]
    assert f.shared_ntok.min() >= 20 and f.shared_ntok.max() <= 70
    assert f.sfx_ntok.min() >= 5 and f.sfx_ntok.max() <= 40


def test_punch_holes_and_lowest_mass():
    w = workloads.make_from_segments("x", 2, 1, 64, [100, 10], [[0, 1], [0, 1]], seed=3)
    idx = workloads.lowest_mass_pages(np.array([5, 1, 3, 1, 9, 0.5, 7]), 0.5)
    assert idx.tolist() == [1, 3, 5]   # ties -> lower index first, floor(0.5*7)=3
    h = workloads.punch_holes(w, 0, idx)
    t = h.tables
    assert t.seg_block_off.tolist() == [0, 4, 5]
    assert t.seg_num_tokens.tolist() == [100 - 48, 10]
    keep = [0, 2, 4, 6]
    assert t.seg_blocks[:4].tolist() == w.tables.seg_blocks[keep].tolist()
    # removing the partial last page leaves only full pages
    h2 = workloads.punch_holes(w, 0, np.array([6]))
    assert h2.tables.seg_num_tokens[0] == 96


def test_unique_and_duplicated_bytes():
    w = workloads.make_tiny()
    assert workloads.unique_kv_bytes(w.layout, w.tables) == 384 * 512       # 192 KiB
    assert workloads.duplicated_kv_bytes(w.layout, w.tables) == 1152 * 512  # 576 KiB
