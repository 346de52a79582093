"""Pins for the CGEE oracle (Section 2.3: Eq. 3-5, Algorithm 3)."""
import numpy as np
import scipy.special
import scipy.stats

import oracle
from helpers import golden_facts


def test_entropy_closed_forms():
    V, D = 1000, 16
    # h = 0: uniform distribution -> H = log V, top-1 = 1 / V
    H, top1 = oracle.logit_entropy(np.zeros((2, D)), np.random.default_rng(0).standard_normal((V, D)))
    assert np.allclose(H, np.log(V), atol=1e-12) and np.allclose(top1, 1.0 / V, atol=1e-15)
    # one huge logit: H -> 0, top-1 -> 1
    w = np.zeros((V, D))
    w[7, 0] = 1.0
    H, top1 = oracle.logit_entropy(np.array([[200.0] + [0.0] * (D - 1)]), w)
    assert H[0] < 1e-80 and top1[0] == 1.0
    # two equal logits far above the rest: H = log 2, top-1 = 1/2
    w[9, 0] = 1.0
    H, top1 = oracle.logit_entropy(np.array([[200.0] + [0.0] * (D - 1)]), w)
    assert abs(H[0] - np.log(2)) < 1e-12 and abs(top1[0] - 0.5) < 1e-12
    # k logits at a, the other V - k at 0: closed form
    k, a = 13, 2.5
    w = np.zeros((V, D))
    w[:k, 0] = a
    H, top1 = oracle.logit_entropy(np.array([[1.0] + [0.0] * (D - 1)]), w)
    Z = k * np.exp(a) + (V - k)
    assert abs(H[0] - (np.log(Z) - k * np.exp(a) * a / Z)) < 1e-12
    assert abs(top1[0] - np.exp(a) / Z) < 1e-15


def test_entropy_against_scipy_and_invariances():
    rng = np.random.default_rng(1)
    B, D, V = 5, 48, 3000
    h, w = rng.standard_normal((B, D)), rng.standard_normal((V, D)) * 0.4
    H, top1 = oracle.logit_entropy(h, w)
    p = scipy.special.softmax(h @ w.T, axis=1)
    assert np.allclose(H, scipy.stats.entropy(p, axis=1), atol=1e-12)
    assert np.allclose(top1, p.max(axis=1), atol=1e-15)
    # a constant added to every logit (one more hidden dimension that multiplies a column of ones) changes nothing
    h2 = np.concatenate([h, np.full((B, 1), 3.0)], axis=1)
    w2 = np.concatenate([w, np.ones((V, 1))], axis=1)
    H2, t2 = oracle.logit_entropy(h2, w2)
    assert np.allclose(H2, H, atol=1e-10) and np.allclose(t2, top1, atol=1e-12)
    # permuting the vocabulary changes nothing; transposed operands would not even have the shape
    perm = rng.permutation(V)
    H3, _ = oracle.logit_entropy(h, w[perm])
    assert np.allclose(H3, H, atol=1e-12)
    # scaling h sharpens the distribution: entropy falls
    H4, _ = oracle.logit_entropy(3.0 * h, w)
    assert np.all(H4 < H)


def test_exit_test_of_algorithm_3():
    f = golden_facts()
    theta, eps, l_min = float(f["cgee_theta_qwen"]), float(f["cgee_eps"]), int(f["cgee_l_min"])
    H = np.array([7.9, 8.0, 7.0, 7.0, 2.0])
    Hp = np.array([7.0, 7.5, 10.1, 9.9, np.inf])
    # H < theta strictly; |dH| < eps strictly; the first layer (H_prev = +inf) never exits
    assert oracle.entropy_exit(H, Hp, 5, l_min, theta, eps).tolist() == [True, False, False, True, False]
    assert oracle.entropy_exit(H, Hp, 1, l_min, theta, eps).tolist() == [False] * 5          # l < l_min
    assert oracle.entropy_exit(H, Hp, 2, l_min, theta, eps).tolist() == [True, False, False, True, False]


def test_level_1_gate_and_confidence():
    f = golden_facts()
    tau, r = float(f["cgee_tau_conf"]), float(f["cgee_r_gap"])
    assert oracle.generation_confidence([[0.5, 1.0], [0.7, 0.0]]).tolist() == [0.6, 0.5]
    assert oracle.verify_skip([0.9, 0.5, 0.8], tau, r)             # gap (0.9 - 0.8) / 0.9 = 0.111
    assert not oracle.verify_skip([0.9, 0.5, 0.86], tau, r)        # gap 0.044 < 0.06: a close competitor
    assert not oracle.verify_skip([0.6, 0.1, 0.2], tau, r)         # a large gap at low confidence
    assert oracle.verify_skip([0.5, 0.375], 0.5, 0.25)             # both thresholds met with equality: >= on both
    assert not oracle.verify_skip([0.5, 0.376], 0.5, 0.25)
    assert not oracle.verify_skip([0.499, 0.1], 0.5, 0.25)
    assert oracle.verify_skip([0.75], tau, r) and not oracle.verify_skip([0.5], tau, r)
    assert not oracle.verify_skip([], tau, r)
    # the order of the branches does not matter
    assert oracle.verify_skip([0.8, 0.9, 0.5], tau, r) == oracle.verify_skip([0.9, 0.5, 0.8], tau, r)
