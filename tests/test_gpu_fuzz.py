"""Seeded random segment structures through the attention path against the oracle.

Each case draws heads (Hkv in 1..8, group size 1..8), head_dim 64 or 128, up to 39 branches, up to
three shared segments with random sharer sets and a private segment per branch, token counts either
uniform or from a list of values around the page, slot and tile sizes (1, 15, 16, 17, ..., 257), and
a query gain of 1, 3 or 8 (sharper softmax).  Both kernels, every row-count class and ragged last
pages come up; outputs and block masses must meet the path's tolerances in every case.
"""
import numpy as np
import pytest

import workloads
from helpers import check_attention, oracle_attention

pytestmark = pytest.mark.gpu

EDGE = [1, 2, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129, 255, 256, 257]


def _case(seed):
    rng = np.random.default_rng(seed)
    hd = int(rng.choice([64, 128, 128, 128]))
    Hkv = int(rng.choice([1, 2, 4, 8]))
    G = int(rng.choice([1, 2, 4, 7, 8]))
    B = int(rng.integers(1, 40))
    seg_ntok, br = [], [[] for _ in range(B)]
    for s in range(int(rng.integers(0, 4))):
        seg_ntok.append(int(rng.choice(EDGE)) if rng.random() < 0.5 else int(rng.integers(1, 700)))
        for b in rng.choice(B, size=int(rng.integers(1, B + 1)), replace=False):
            br[int(b)].append(s)
    for b in range(B):
        if rng.random() < 0.85 or not br[b]:
            n = int(rng.choice(EDGE)) if rng.random() < 0.5 else int(rng.integers(0, 300))
            if n == 0 and not br[b] and rng.random() < 0.7:
                n = 5
            seg_ntok.append(n)
            br[b].append(len(seg_ntok) - 1)
        br[b] = sorted(br[b])
    gain = float(rng.choice([1.0, 1.0, 3.0, 8.0]))
    return workloads.make_from_segments(f"fuzz{seed}", Hkv * G, Hkv, hd, seg_ntok, br, seed=1000 + seed, q_gain=gain)


@pytest.mark.parametrize("first", [0, 40, 80])
def test_random_segment_structures_match_the_oracle(first):
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    for seed in range(first, first + 40):
        w = _case(seed)
        plan = rk.rksc_plan_create(w.layout, w.tables)
        out, mass, status = rk.rksc_branch_decode_attention(plan, w.q.to(dev), w.k_pool.to(dev), w.v_pool.to(dev))
        torch.cuda.synchronize()
        assert int(status.item()) == 0, seed
        ref_out, ref_m = oracle_attention(w)
        try:
            check_attention(out.cpu().numpy(), rk.split_block_mass(plan, mass), ref_out, ref_m)
        except AssertionError as e:
            raise AssertionError(f"seed {seed}: {e}") from None


def test_random_gate_shapes_match_the_oracle():
    """The gate over random shapes (1-69 branches, 1-8 roots, 1-40 layers, hidden sizes from 1 to 4097
    including ones that are no multiple of four), random perturbation levels, alpha and tau from the
    paper's grids, now and then a zero-norm layer vector: map bit-exact wherever the oracle's sigma
    keeps 1e-3 clear of tau, sigma within 2e-5."""
    import torch
    import oracle
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    checked = 0
    for trial in range(90):
        rng = np.random.default_rng(trial)
        B, P, L = int(rng.integers(1, 70)), int(rng.integers(1, 9)), int(rng.integers(1, 41))
        D = int(rng.choice([1, 3, 4, 7, 64, 100, 255, 256, 1000, 1024, 3584, 4096, 4097]))
        cand = rng.integers(0, P, size=B).astype(np.int32)
        eps = [float(rng.choice([0.0, 0.1, 0.203, 0.5, 0.75, 1.5, np.inf])) for _ in range(B)]
        alpha = float(rng.choice([0.0, 0.5, 1.0, 1.5, 2.0]))
        tau = float(rng.choice([0.0, 0.5, 0.82, 0.9, 0.95]))
        g = workloads.make_gate_inputs(cand, P, L, D, eps, alpha=alpha, tau=tau, seed=trial)
        hb = g.h_branch.clone()
        if trial % 9 == 0:
            hb[0, 0] = 0.0
        m_ref, s_ref = oracle.asks_gate(hb.numpy(), g.h_root.numpy(), cand, alpha, tau)
        if np.abs(s_ref - np.float32(tau)).min() < 1e-3:
            continue
        m, s = rk.rksc_asks_gate(hb.to(dev), g.h_root.to(dev), torch.from_numpy(cand).to(dev), alpha, tau)
        torch.cuda.synchronize()
        assert np.array_equal(m.cpu().numpy(), m_ref), trial
        assert np.abs(s.cpu().numpy() - s_ref).max() <= 2e-5, trial
        checked += 1
    assert checked >= 60


def test_random_eviction_problems_match_algorithm_4():
    """RSBCM selection on random scores and depths (sizes around the kernel's 32 / 256 / 1024 boundaries,
    capacities from 0 to more than n, with and without ties) against the oracle that evicts the arg-min
    one entry at a time: the same entries, bit for bit."""
    import torch
    import oracle
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    for trial in range(70):
        rng = np.random.default_rng(trial)
        n = int(rng.choice([1, 2, 7, 31, 32, 33, 255, 256, 257, 700, 1023, 1024, 1025]))
        cap = int(rng.integers(0, n + 2))
        score, depth = workloads.make_eviction_inputs(n, seed=trial, tie_levels=int(rng.choice([0, 0, 2, 5, 50])))
        ref = oracle.rsbcm_evict(score, depth, cap)[0]
        ev, cnt = rk.rksc_rsbcm_evict(torch.from_numpy(score).to(dev), torch.from_numpy(depth).to(dev), cap)
        torch.cuda.synchronize()
        assert np.array_equal(ev.cpu().numpy().astype(bool), ref), (trial, n, cap)
        assert int(cnt.item()) == int(ref.sum()), (trial, n, cap)


def test_random_unembedding_shapes_match_the_entropy_oracle():
    """Entropy and top-1 probability of softmax(h W_u^T) over random shapes (1-32 rows, vocabularies from
    1 to 50257 entries around the 128-row tile, flat and peaked logits)."""
    import torch
    import oracle
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    for trial in range(20):
        rng = np.random.default_rng(100 + trial)
        B = int(rng.integers(1, 33))
        D = int(rng.choice([64, 128, 512, 1000, 3584]))
        V = int(rng.choice([1, 5, 127, 128, 129, 1000, 32000, 50257]))
        h, w = workloads.make_cgee_inputs(B, D, V, seed=trial, logit_std=float(rng.choice([0.5, 3.0, 8.0])))
        H_ref, p_ref = oracle.logit_entropy(oracle.to_f32_numpy(h), oracle.to_f32_numpy(w))
        H, p, status = rk.rksc_cgee_logit_entropy(h.to(dev), w.to(dev))[:3]
        torch.cuda.synchronize()
        assert int(status.item()) == 0, trial
        assert np.abs(H.cpu().numpy() - H_ref).max() <= 2e-3, (trial, B, D, V)
        assert (np.abs(p.cpu().numpy() - p_ref) / p_ref).max() <= 2e-3, (trial, B, D, V)


def test_random_suffix_prefill_problems_match_the_oracle():
    """Suffix prefill (s in 1..16 query tokens per branch, causal inside the suffix) over random shared /
    private segment structures whose last segment holds s tokens or a few more: the library's
    virtual-branch tables bit-exact against the oracle's, outputs and masses within the tolerances."""
    from test_gpu_suffix_prefill import _run

    edge = [1, 2, 15, 16, 17, 31, 32, 33, 63, 64, 65, 127, 128, 129]
    for seed in range(60):
        rng = np.random.default_rng(seed)
        s = int(rng.choice([1, 2, 3, 5, 8, 16]))
        hd, Hkv, G = int(rng.choice([64, 128, 128])), int(rng.choice([1, 2, 4])), int(rng.choice([1, 4, 7]))
        B = int(rng.integers(1, 12))
        seg_ntok, br = [], [[] for _ in range(B)]
        for sh in range(int(rng.integers(0, 3))):
            seg_ntok.append(int(rng.choice(edge)) if rng.random() < 0.5 else int(rng.integers(1, 400)))
            for b in rng.choice(B, size=int(rng.integers(1, B + 1)), replace=False):
                br[int(b)].append(sh)
        for b in range(B):
            extra = int(rng.choice([0, 1, 15, 16, 17])) if rng.random() < 0.6 else int(rng.integers(0, 120))
            seg_ntok.append(s + extra)
            br[b] = sorted(br[b]) + [len(seg_ntok) - 1]
        w = workloads.make_from_segments(f"pf{seed}", Hkv * G, Hkv, hd, seg_ntok, br, seed=3000 + seed)
        try:
            _run(w, s, seed=seed)
        except AssertionError as e:
            raise AssertionError(f"seed {seed} (s = {s}): {e}") from None
