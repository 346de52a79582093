"""RSBCM eviction on the GPU vs the fp64 oracle (Section 2.4, Algorithm 4): bit-exact scores and
selection on the same seeded inputs; the chain attention -> scores -> eviction -> holed attention."""
import numpy as np
import pytest

import oracle
import workloads
from helpers import check_attention, cuda_attention, oracle_attention, oracle_gate, oracle_tables_from_map

pytestmark = pytest.mark.gpu


def _pack(plan, masses, Hq):
    """Per-branch [Hq][nblk] arrays -> the flat block_mass layout of the library."""
    import torch
    flat = np.zeros(max(1, plan.mass_elems), dtype=np.float32)
    mo = plan.mass_off
    for b, m in enumerate(masses):
        flat[int(mo[b]) * Hq:int(mo[b + 1]) * Hq] = np.asarray(m, np.float32).reshape(-1)
    return torch.from_numpy(flat).to("cuda:0")


def _gate_tables(w):
    """Tables of an end-to-end workload: from the oracle's gate map."""
    d = oracle_tables_from_map(w, oracle_gate(w.gate)[0])
    return workloads.Tables(**{k: np.asarray(v, np.int32) for k, v in d.items()})


def _gpu_scores(w, masses, tables=None):
    import torch
    import paper_2606_09937_b200 as rk
    t = tables if tables is not None else w.tables
    plan = rk.rksc_plan_create(w.layout, t)
    sc = rk.rksc_rsbcm_page_scores(plan, _pack(plan, masses, w.layout.num_q_heads))
    torch.cuda.synchronize()
    return sc.cpu().numpy(), plan


def _oracle_scores(w, masses, tables=None):
    t = tables if tables is not None else w.tables
    return oracle.page_scores(t.seg_block_off, t.br_seg_off, t.br_segs, masses, w.layout.num_q_heads)


def _gpu_evict(score, depth, cap):
    import torch
    import paper_2606_09937_b200 as rk
    ev, cnt = rk.rksc_rsbcm_evict(torch.from_numpy(np.asarray(score, np.float64)).to("cuda:0"),
                                  torch.from_numpy(np.asarray(depth, np.int32)).to("cuda:0"), cap)
    torch.cuda.synchronize()
    return ev.cpu().numpy().astype(bool), int(cnt.item())


@pytest.mark.parametrize("name", ["tiny", "tot_small", "dup_segment", "serving_small", "holes"])
def test_page_scores_bit_exact(name):
    if name == "tiny":
        w = workloads.make_tiny()
    elif name == "tot_small":
        w = workloads.make_tot(root_tokens=700, level_tokens=90, branching=3, depth=2)
    elif name == "dup_segment":
        # a branch listing one segment twice, an empty segment, a segment nobody lists
        w = workloads.make_from_segments("dup", 8, 2, 64, [37, 0, 100, 16, 5], [[0, 0, 2], [2, 1, 3], [3], []], seed=21)
    elif name == "serving_small":
        w = workloads.make_batched_serving(problems=3, branches_per=40, prefix_range=(900, 1300),
                                           suffix_range=(40, 90))
        w.tables = _gate_tables(w)
    else:
        w = workloads.punch_holes(workloads.make_tiny(), 0, np.array([1, 5, 15]))
    masses = workloads.make_block_masses(w.tables, w.layout.num_q_heads)
    got, plan = _gpu_scores(w, masses)
    ref = _oracle_scores(w, masses)
    assert got.shape == ref.shape and np.array_equal(got, ref)
    assert abs(ref.sum() - sum(float(np.asarray(m, np.float64).sum()) for m in masses)) < 1e-6


def test_paper_stress_case():
    # N_max = 4 with 8 cached entries: exactly 4 evictions (Appendix, deep-tree validation)
    score, depth = workloads.make_eviction_inputs(8)
    ev, cnt = _gpu_evict(score, depth, 4)
    ref, _ = oracle.rsbcm_evict(score, depth, 4)
    assert cnt == 4 and int(ev.sum()) == 4 and np.array_equal(ev, ref)
    ev, cnt = _gpu_evict(score, depth, 2000)      # the default capacity: nothing to do
    assert cnt == 0 and not ev.any()


@pytest.mark.parametrize("n", [1, 2, 31, 1023, 1024, 1025, 2500])
@pytest.mark.parametrize("ties", [0, 5])
def test_evict_matches_the_literal_loop(n, ties):
    score, depth = workloads.make_eviction_inputs(n, seed=100 + n, tie_levels=ties)
    for cap in sorted({0, 1, n // 3, n - 1, n, n + 7}):
        ev, cnt = _gpu_evict(score, depth, cap)
        ref, order = oracle.rsbcm_evict(score, depth, cap)
        assert cnt == len(order) == max(0, n - cap)
        assert np.array_equal(ev, ref), (n, ties, cap)


def test_evict_edge_values():
    # zeros of both signs tie; equal omega from different (score, depth) pairs tie; index decides
    score = np.array([0.0, -0.0, 6.0, 2.0, 3.0, 0.0])
    depth = np.array([3, 0, 5, 1, 2, 9], np.int32)        # omega: 0, 0, 1, 1, 1, 0
    for cap in range(0, 7):
        ev, _ = _gpu_evict(score, depth, cap)
        ref, _ = oracle.rsbcm_evict(score, depth, cap)
        assert np.array_equal(ev, ref), cap
    # n = 0
    import torch
    import paper_2606_09937_b200 as rk
    ev, cnt = rk.rksc_rsbcm_evict(torch.empty(0, dtype=torch.float64, device="cuda:0"),
                                  torch.empty(0, dtype=torch.int32, device="cuda:0"), 4)
    torch.cuda.synchronize()
    assert ev.numel() == 0 and int(cnt.item()) == 0


@pytest.mark.parametrize("n,ties", [(200_000, 0), (200_000, 40), (1_000_003, 0)])
def test_evict_large_by_properties(n, ties):
    # too large for the literal loop: the marked set must be the k smallest by (omega, index),
    # which the CPU tests show to be what the loop ends with
    score, depth = workloads.make_eviction_inputs(n, seed=7, tie_levels=ties)
    cap = n // 2 + 3
    ev, cnt = _gpu_evict(score, depth, cap)
    k = n - cap
    assert cnt == k and int(ev.sum()) == k
    omega = score / (depth + 1).astype(np.float64)
    hi = omega[ev].max()
    assert hi <= omega[~ev].min()
    # among entries equal to the largest evicted omega, the evicted ones come first
    tie = np.flatnonzero(omega == hi)
    flags = ev[tie]
    assert not np.any(~flags[:-1] & flags[1:])


def test_chain_attention_scores_eviction_holed_attention():
    import torch
    import paper_2606_09937_b200 as rk
    w = workloads.make_tot(root_tokens=900, level_tokens=130, branching=3, depth=2)
    t = w.tables
    Hq = w.layout.num_q_heads
    # oracle chain
    ref_out, ref_m = oracle_attention(w)
    sc_ref = oracle.page_scores(t.seg_block_off, t.br_seg_off, t.br_segs, ref_m, Hq)
    # depth of a segment = its position on a root-to-leaf path
    seg_depth = np.zeros(len(t.seg_num_tokens), np.int32)
    for b in range(t.num_branches):
        for pos, s in enumerate(t.br_segs[t.br_seg_off[b]:t.br_seg_off[b + 1]]):
            seg_depth[s] = pos
    depth = np.repeat(seg_depth, np.diff(t.seg_block_off)).astype(np.int32)
    n = sc_ref.shape[0]
    omega_ref = sc_ref / (depth + 1)
    k = n // 3
    cap = n - k
    ev_ref, _ = oracle.rsbcm_evict(sc_ref, depth, cap)
    holed_ref = oracle.apply_eviction(t.seg_block_off, t.seg_blocks, t.seg_num_tokens, ev_ref)
    # CUDA chain
    out, m, plan = cuda_attention(w)
    check_attention(out, m, ref_out, ref_m)
    sc, _ = _gpu_scores(w, m)
    score_tol = 1e-4 * t.num_branches * Hq          # the masses' tolerance, summed over every (b, h)
    assert np.abs(sc - sc_ref).max() < score_tol
    ev, cnt = _gpu_evict(sc, depth, cap)
    assert cnt == k and int(ev.sum()) == k
    # the masses differ within their tolerance, so entries whose omega lies that close to the
    # k-th smallest may legitimately fall on either side; every other entry must agree
    kth = np.sort(omega_ref)[k - 1]
    diff = np.flatnonzero(ev != ev_ref)
    assert np.all(np.abs(omega_ref[diff] - kth) <= 2 * score_tol / (depth[diff] + 1))
    assert len(diff) <= n // 20
    holed = rk.rksc_tables_drop_evicted(t, ev)
    assert int(holed.seg_block_off[-1]) == n - k
    holed = rk.rksc_tables_drop_evicted(t, ev_ref)
    assert holed.seg_block_off.tolist() == holed_ref[0].tolist()
    assert holed.seg_blocks.tolist() == holed_ref[1].tolist()
    assert holed.seg_num_tokens.tolist() == holed_ref[2].tolist()
    ht = workloads.Tables(seg_block_off=holed_ref[0], seg_blocks=holed_ref[1], seg_num_tokens=holed_ref[2],
                          br_seg_off=t.br_seg_off, br_segs=t.br_segs)
    ref_out2, ref_m2 = oracle_attention(w, ht)
    out2, m2, _ = cuda_attention(w, holed)
    check_attention(out2, m2, ref_out2, ref_m2)


def test_full_size_scores_batched_serving():
    # the bench's configuration: every entry, bit for bit, on synthetic masses
    w = workloads.make_batched_serving()
    w.tables = _gate_tables(w)
    masses = workloads.make_block_masses(w.tables, w.layout.num_q_heads)
    got, plan = _gpu_scores(w, masses)
    ref = _oracle_scores(w, masses)
    assert np.array_equal(got, ref)
    depth = np.zeros(got.shape[0], np.int32)
    ev, cnt = _gpu_evict(got, depth, 2000)
    assert cnt == got.shape[0] - 2000
    kth = np.sort(ref)[cnt - 1]
    assert ev[ref < kth].all() and not ev[ref > kth].any()
