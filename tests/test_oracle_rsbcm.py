"""Pins for the RSBCM oracle (Section 2.4, Algorithm 4)."""
import numpy as np

import oracle
import workloads
from helpers import golden_facts, oracle_attention


def test_paper_stress_case_exactly_b_minus_nmax_evictions():
    facts = golden_facts()
    B, nmax = int(facts["branches_per_problem"]), int(facts["rsbcm_stress_capacity"])
    rng = np.random.default_rng(0)
    ev, order = oracle.rsbcm_evict(rng.random(B), np.zeros(B, int), nmax)
    assert int(ev.sum()) == len(order) == B - nmax == int(facts["rsbcm_stress_evictions_per_solve"])
    ev, order = oracle.rsbcm_evict(rng.random(B), np.zeros(B, int), B)       # at capacity: dormant
    assert not ev.any() and len(order) == 0
    ev, _ = oracle.rsbcm_evict(rng.random(B), np.zeros(B, int), 2000)        # the default capacity: dormant
    assert not ev.any()


def test_ascending_omega_depth_discount_and_ties():
    # omega = score / (depth + 1): hand values
    score = np.array([6.0, 6.0, 1.0, 9.0, 2.0])
    depth = np.array([0, 2, 0, 8, 1])
    # omega = 6, 2, 1, 1, 1 -> ascending with ties broken by position: entries 2, 3, 4, then 1
    ev, order = oracle.rsbcm_evict(score, depth, 1)
    assert order.tolist() == [2, 3, 4, 1] and ev.tolist() == [False, True, True, True, True]
    # equal scores: deeper blocks go first
    ev, order = oracle.rsbcm_evict(np.ones(4), np.array([0, 3, 1, 2]), 1)
    assert order.tolist() == [1, 3, 2]
    # equal depth: lowest score goes first
    ev, order = oracle.rsbcm_evict(np.array([0.3, 0.1, 0.2]), np.zeros(3, int), 0)
    assert order.tolist() == [1, 2, 0]


def test_loop_equals_k_smallest_by_omega_then_index():
    rng = np.random.default_rng(1)
    for _ in range(20):
        n = int(rng.integers(1, 60))
        score = rng.integers(0, 6, n).astype(np.float64) / 4        # many ties
        depth = rng.integers(0, 4, n)
        cap = int(rng.integers(0, n + 2))
        ev, order = oracle.rsbcm_evict(score, depth, cap)
        omega = score / (depth + 1)
        ref = sorted(range(n), key=lambda i: (omega[i], i))[: max(0, n - cap)]
        assert order.tolist() == ref and sorted(np.flatnonzero(ev).tolist()) == sorted(ref)


def test_page_scores_sum_and_sharing():
    w = workloads.make_tot(head_dim=64, num_q_heads=4, num_kv_heads=2, root_tokens=50, level_tokens=21,
                           branching=2, depth=2)
    t = w.tables
    _, masses = oracle_attention(w)
    sc = oracle.page_scores(t.seg_block_off, t.br_seg_off, t.br_segs, masses, 4)
    assert sc.shape[0] == int(t.seg_block_off[-1]) and (sc >= 0).all()
    # every (branch, head) spreads a mass of exactly 1 over the entries it attends to
    assert abs(sc.sum() - t.num_branches * 4) < 1e-10
    # brute force for one entry: page 1 of the root segment is read by all 4 leaves
    e = int(t.seg_block_off[0]) + 1
    assert abs(sc[e] - sum(m[:, 1].sum() for m in masses)) < 1e-12
    # an entry of a leaf segment is read by that leaf only, at the right logical offset
    leaf_seg = int(t.br_segs[t.br_seg_off[3 + 1] - 1])
    loff = sum(int(t.seg_block_off[s + 1] - t.seg_block_off[s]) for s in t.br_segs[t.br_seg_off[3]:t.br_seg_off[4] - 1])
    assert abs(sc[int(t.seg_block_off[leaf_seg])] - masses[3][:, loff].sum()) < 1e-12
    # a segment nobody lists scores 0
    w2 = workloads.make_tiny()
    _, m2 = oracle_attention(w2)
    sc2 = oracle.page_scores(w2.tables.seg_block_off, w2.tables.br_seg_off, w2.tables.br_segs, m2, 8)
    lo, hi = int(w2.tables.seg_block_off[1]), int(w2.tables.seg_block_off[2])     # the unused private copy
    assert np.all(sc2[lo:hi] == 0) and abs(sc2.sum() - 4 * 8) < 1e-10


def test_apply_eviction_hand_case_and_hole_puncher():
    # one segment of 3 pages holding 40 tokens (16 + 16 + 8), one of 1 page holding 5
    off, blocks, ntok = np.array([0, 3, 4]), np.array([7, 3, 9, 2]), np.array([40, 5])
    o, b, n = oracle.apply_eviction(off, blocks, ntok, np.array([0, 1, 0, 0], bool))
    assert o.tolist() == [0, 2, 3] and b.tolist() == [7, 9, 2] and n.tolist() == [24, 5]
    o, b, n = oracle.apply_eviction(off, blocks, ntok, np.array([0, 0, 1, 1], bool))      # partial tail pages go
    assert o.tolist() == [0, 2, 2] and b.tolist() == [7, 3] and n.tolist() == [32, 0]
    o, b, n = oracle.apply_eviction(off, blocks, ntok, np.zeros(4, bool))
    assert o.tolist() == off.tolist() and b.tolist() == blocks.tolist() and n.tolist() == ntok.tolist()
    # against the workload generator's hole puncher, one segment at a time
    w = workloads.make_tiny()
    t = w.tables
    rng = np.random.default_rng(3)
    ev = rng.random(int(t.seg_block_off[-1])) < 0.4
    o, b, n = oracle.apply_eviction(t.seg_block_off, t.seg_blocks, t.seg_num_tokens, ev)
    w2 = w
    for s in range(len(t.seg_num_tokens)):
        lo, hi = int(t.seg_block_off[s]), int(t.seg_block_off[s + 1])
        w2 = workloads.punch_holes(w2, s, np.flatnonzero(ev[lo:hi]))
    assert o.tolist() == w2.tables.seg_block_off.tolist() and b.tolist() == w2.tables.seg_blocks.tolist()
    assert n.tolist() == w2.tables.seg_num_tokens.tolist()
