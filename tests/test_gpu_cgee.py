"""CGEE numerics on the GPU vs the fp64 oracle (Section 2.3: Eq. 3-5, Algorithm 3)."""
import numpy as np
import pytest

import oracle
import workloads
from helpers import golden_facts

pytestmark = pytest.mark.gpu

# bf16 x bf16 products are exact in fp32; what differs from the oracle is the fp32 accumulation over D
# (relative 2^-24 * sqrt(D) of |z| ~ 10: ~1e-5 per logit) and the fp32 softmax statistics over V terms.
H_ATOL = 2e-3          # nats
P_RTOL = 2e-3          # relative, top-1 probability


def _run(B, D, V, seed, peaked=()):
    import torch
    import paper_2606_09937_b200 as rk
    h, w = workloads.make_cgee_inputs(B, D, V, seed=seed, peaked_rows=peaked)
    H, top1, status = rk.rksc_cgee_logit_entropy(h.to("cuda:0"), w.to("cuda:0"))
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    ref_H, ref_top1 = oracle.logit_entropy(oracle.to_f32_numpy(h), oracle.to_f32_numpy(w))
    H, top1 = H.cpu().numpy().astype(np.float64), top1.cpu().numpy().astype(np.float64)
    assert np.abs(H - ref_H).max() <= H_ATOL, (H, ref_H)
    assert np.abs(top1 / ref_top1 - 1).max() <= P_RTOL, (top1, ref_top1)
    return H, top1, ref_H


@pytest.mark.parametrize("B,D,V", [(1, 64, 128), (8, 256, 5000), (16, 3584, 9000), (5, 1000, 129), (3, 72, 127),
                                   (20, 512, 3000), (40, 128, 1000)])
def test_entropy_and_top1(B, D, V):
    # one tile and less, ragged last tile, D not a multiple of 64, more rows than one launch takes
    H, top1, ref = _run(B, D, V, seed=100 + B, peaked=(0,) if B > 2 else ())
    assert np.all(H >= -1e-6) and np.all(H <= np.log(V) + 1e-4)


def test_closed_forms_on_device():
    import torch
    import paper_2606_09937_b200 as rk
    V, D = 1000, 64
    w = torch.randn((V, D), generator=torch.Generator().manual_seed(1)).to(torch.bfloat16)
    h = torch.zeros((2, D), dtype=torch.bfloat16)
    H, top1, _ = rk.rksc_cgee_logit_entropy(h.cuda(), w.cuda())
    assert np.allclose(H.cpu().numpy(), np.log(V), atol=1e-5) and np.allclose(top1.cpu().numpy(), 1.0 / V, rtol=1e-5)
    # one logit far above the rest: entropy ~ 0, top-1 ~ 1
    w2 = torch.zeros((V, D), dtype=torch.bfloat16)
    w2[7, 0] = 1.0
    h2 = torch.zeros((1, D), dtype=torch.bfloat16)
    h2[0, 0] = 100.0
    H, top1, _ = rk.rksc_cgee_logit_entropy(h2.cuda(), w2.cuda())
    assert abs(float(H[0])) < 1e-6 and abs(float(top1[0]) - 1.0) < 1e-6


def test_vocabulary_sized_like_the_paper_models():
    # Qwen2.5-7B: D = 3584, V = 152064 (Section 3, models); B = 8 branches
    H, top1, ref = _run(8, 3584, 152064, seed=5, peaked=(3,))
    assert top1[3] > 0.3                                            # the aligned row has a dominant token


def test_exit_test_and_level_1_gate():
    import torch
    import paper_2606_09937_b200 as rk
    f = golden_facts()
    theta, eps, l_min = float(f["cgee_theta_qwen"]), float(f["cgee_eps"]), int(f["cgee_l_min"])
    H = np.array([7.9, 8.0, 7.0, 7.0, 2.0, 7.5], np.float32)
    Hp = np.array([7.0, 7.5, 10.1, 9.9, np.inf, 7.5], np.float32)
    for layer in (1, 2, 5):
        got = rk.rksc_cgee_entropy_exit(torch.from_numpy(H).cuda(), torch.from_numpy(Hp).cuda(), layer, l_min, theta, eps)
        ref = oracle.entropy_exit(H, Hp, layer, l_min, np.float32(theta), np.float32(eps))
        assert got.cpu().numpy().astype(bool).tolist() == ref.tolist()
    tau, r = float(f["cgee_tau_conf"]), float(f["cgee_r_gap"])
    rng = np.random.default_rng(4)
    for case in range(30):
        B, t = int(rng.integers(1, 40)), int(rng.integers(1, 33))
        steps = rng.uniform(0.2, 1.0, (t, B)).astype(np.float32)
        if case % 3 == 0:
            steps[:, 0] = 0.97                                   # a clear winner
        conf, skip = rk.rksc_cgee_verify_skip(torch.from_numpy(steps).cuda(), tau, r)
        ref_p = oracle.generation_confidence(steps)
        assert np.abs(conf.cpu().numpy() - ref_p).max() < 1e-6
        srt = np.sort(ref_p)[::-1]
        gap = (srt[0] - (srt[1] if B > 1 else 0.0)) / srt[0]
        if abs(srt[0] - tau) > 1e-5 and abs(gap - r) > 1e-5:     # away from the thresholds the decision is unique
            assert bool(skip.item()) == oracle.verify_skip(ref_p, tau, r), (case, srt[:2])
    # equal leaders: no gap
    steps = np.full((4, 3), 0.9, np.float32)
    _, skip = rk.rksc_cgee_verify_skip(torch.from_numpy(steps).cuda(), tau, r)
    assert int(skip.item()) == 0 and not oracle.verify_skip([0.9, 0.9, 0.9], tau, r)
