"""Pins for the gate oracle: closed forms, brute force, invariants (Eq. 2, Algorithm 2)."""
import math
from decimal import Decimal, getcontext

import numpy as np
import pytest

import oracle
import workloads
from helpers import golden_facts, oracle_gate

getcontext().prec = 50


def test_weights_geometric_closed_form():
    # exp(alpha*l/L) is a geometric sequence with ratio r = exp(alpha/L), so
    # w_l = r^(l-1) (r-1) / (r^L - 1): the normalised geometric series.
    for alpha in golden_facts()["alpha_grid"]:
        for L in (1, 4, 28, 32, 40):
            w = oracle.layer_weights(alpha, L)
            r = Decimal(alpha / L).exp()
            ref = [float(r ** (l - 1) * (r - 1) / (r ** L - 1)) for l in range(1, L + 1)]
            assert np.allclose(w, ref, rtol=1e-13, atol=0)
            assert abs(w.sum() - 1.0) < 1e-14
            assert np.all(np.diff(w) > 0)  # later layers weigh more


def test_weights_printed_values():
    # hand-evaluated softmax of (alpha*l/L): L = 4
    assert np.allclose(oracle.layer_weights(0.5, 4),
                       [0.205248, 0.232576, 0.263543, 0.298633], atol=5e-7)
    assert np.allclose(oracle.layer_weights(1.5, 4),
                       [0.130681, 0.190140, 0.276652, 0.402527], atol=5e-7)
    w = oracle.layer_weights(1.5, 28)
    assert abs(w[-1] / w[0] - math.exp(1.5 * 27 / 28)) < 1e-12


def test_weights_uniform_and_shift_invariance():
    assert np.allclose(oracle.layer_weights(0.0, 7), np.full(7, 1 / 7), atol=1e-16)
    # numbering layers from 0 multiplies every exp by a constant: same weights
    L, alpha = 12, 1.5
    e0 = np.array([math.exp(alpha * l / L) for l in range(0, L)])
    assert np.allclose(oracle.layer_weights(alpha, L), e0 / e0.sum(), rtol=1e-14)


def _rand(shape, seed):
    return np.random.default_rng(seed).standard_normal(shape).astype(np.float32)


def test_sigma_identical_scaled_negated_orthogonal():
    facts = golden_facts()
    L, D = 6, 64
    hr = _rand((1, L, D), 1)
    cand = [0]
    for alpha in (0.5, 1.5):
        _, s = oracle.asks_gate(hr, hr, cand, alpha, 0.5)
        assert abs(s[0] - facts["identical_prefix_sigma"]) < 1e-12
        _, s = oracle.asks_gate(3.7 * hr, hr, cand, alpha, 0.5)
        assert abs(s[0] - 1.0) < 1e-7   # fp32 scaling of the inputs
        m, s = oracle.asks_gate(-hr, hr, cand, alpha, 0.5)
        assert abs(s[0] + 1.0) < 1e-12 and m[0] == -1
    # orthogonal by construction: disjoint supports
    a = np.zeros((1, L, D), np.float32)
    b = np.zeros((1, L, D), np.float32)
    a[..., : D // 2] = _rand((1, L, D // 2), 2)
    b[..., D // 2:] = _rand((1, L, D // 2), 3)
    _, s = oracle.asks_gate(a, b, cand, 1.5, 0.5)
    assert s[0] == 0.0
    # only the last layer orthogonal: sigma = 1 - w_L
    c = hr.copy()
    c[0, L - 1] = 0
    c[0, L - 1, 0] = 1.0
    r = hr.copy()
    r[0, L - 1] = 0
    r[0, L - 1, 1] = 1.0
    _, s = oracle.asks_gate(c, r, cand, 1.5, 0.5)
    assert abs(s[0] - (1.0 - oracle.layer_weights(1.5, L)[-1])) < 1e-12
    # only the FIRST layer orthogonal: catches reversed layer weights
    c = hr.copy(); r = hr.copy()
    c[0, 0] = 0; c[0, 0, 0] = 1.0
    r[0, 0] = 0; r[0, 0, 1] = 1.0
    _, s = oracle.asks_gate(c, r, cand, 1.5, 0.5)
    assert abs(s[0] - (1.0 - oracle.layer_weights(1.5, L)[0])) < 1e-12


def test_sigma_known_angles_per_layer():
    # h_b = cos(t_l) e0 + sin(t_l) e1 against root e0: cosine is cos(t_l) exactly
    L = 5
    thetas = [0.1, 0.7, 1.2, 2.0, 3.0]
    hb = np.zeros((1, L, 8), np.float64)
    hr = np.zeros((1, L, 8), np.float64)
    for l, t in enumerate(thetas):
        hb[0, l, 0], hb[0, l, 1] = 2.5 * math.cos(t), 2.5 * math.sin(t)
        hr[0, l, 0] = 0.3
    w = oracle.layer_weights(1.0, L)
    _, s = oracle.asks_gate(hb, hr, [0], 1.0, 0.0)
    assert abs(s[0] - sum(w[l] * math.cos(t) for l, t in enumerate(thetas))) < 1e-12
    assert -1.0 <= s[0] <= 1.0


def test_sigma_noise_model():
    # h_b = h_r + eps*n with independent n: cos -> 1/sqrt(1+eps^2) for large D
    g = workloads.make_gate_inputs([0, 0], 1, 4, 16384, [workloads.generators.EPS_NEAR,
                                   workloads.generators.EPS_FAR], 0.5, 0.9, seed=5)
    _, s = oracle_gate(g)
    assert abs(s[0] - 1 / math.sqrt(1 + 0.203 ** 2)) < 5e-3
    assert abs(s[1] - 1 / math.sqrt(1 + 0.75 ** 2)) < 1e-2


def _gate_brute(hb, hr, cand, alpha, tau):
    """Independent twin: scalar loops in 50-digit decimal arithmetic."""
    B, L, D = hb.shape
    es = [(Decimal(alpha) * Decimal(l) / Decimal(L)).exp() for l in range(1, L + 1)]
    tot = sum(es)
    sig = []
    for b in range(B):
        r = cand[b]
        s = Decimal(0)
        for l in range(L):
            dot = nb = nr = Decimal(0)
            for k in range(D):
                x = Decimal(float(hb[b, l, k])); y = Decimal(float(hr[r, l, k]))
                dot += x * y; nb += x * x; nr += y * y
            s += es[l] / tot * dot / (nb.sqrt() * nr.sqrt())
        sig.append(float(s))
    return sig


def test_gate_brute_force_twin():
    B, P, L, D = 5, 3, 4, 24
    hb = _rand((B, L, D), 10)
    hr = _rand((P, L, D), 11)
    cand = [2, 0, 1, 1, 2]
    alpha = float(np.float32(1.5))
    _, s = oracle.asks_gate(hb, hr, cand, alpha, 0.1)
    ref = _gate_brute(hb, hr, cand, alpha, 0.1)
    assert np.allclose(s, ref, rtol=0, atol=1e-13)


def test_map_uses_candidate_and_threshold_is_inclusive():
    L, D = 2, 16
    hr = _rand((3, L, D), 20)
    hb = np.stack([hr[2], hr[0], hr[1]])
    m, s = oracle.asks_gate(hb, hr, [2, 0, 1], 1.5, 0.95)
    assert m.tolist() == [2, 0, 1] and np.allclose(s, 1.0)
    m, _ = oracle.asks_gate(hb, hr, [0, 1, 2], 1.5, 0.95)   # wrong candidates: unrelated roots
    assert m.tolist() == [-1, -1, -1]
    # sigma exactly 0.5: alpha = 0 (uniform weights), layer 1 identical, layer 2 orthogonal
    a = np.zeros((1, 2, 4)); r = np.zeros((1, 2, 4))
    a[0, 0, 0] = 1; r[0, 0, 0] = 1; a[0, 1, 0] = 1; r[0, 1, 1] = 1
    m, s = oracle.asks_gate(a, r, [0], 0.0, 0.5)
    assert s[0] == 0.5 and m[0] == 0            # sigma >= tau shares
    m, _ = oracle.asks_gate(a, r, [0], 0.0, float(np.nextafter(np.float32(0.5), np.float32(1))))
    assert m[0] == -1


def test_tau_zero_shares_everything_with_nonnegative_cosines():
    # tau = 0 is the paper's "vLLM-equivalent" unconditional reuse in the identical-prefix regime
    g = workloads.make_gate_inputs([0] * 6, 1, 4, 512, [0.0, 0.2, 0.5, 0.75, 1.0, 1.5], 1.5, 0.0, seed=6)
    m, s = oracle_gate(g)
    assert (s > 0).all() and (m == 0).all()


def test_zero_norm_and_nan():
    L, D = 3, 8
    hr = _rand((1, L, D), 30)
    hb = hr.copy()
    hb[0, 1] = 0
    w = oracle.layer_weights(1.5, L)
    _, s = oracle.asks_gate(hb, hr, [0], 1.5, 0.5)
    assert abs(s[0] - (1 - w[1])) < 1e-12
    hb[0, 2, 0] = np.nan
    m, s = oracle.asks_gate(hb, hr, [0], 1.5, -1.0)
    assert m[0] == -1 and math.isnan(s[0])


@pytest.mark.parametrize("name", ["tiny", "qwen_layer"])
def test_config_gate_margin(name):
    w = workloads.make_config(name)
    m, s = oracle_gate(w.gate)
    tau = float(np.float32(w.gate.tau))
    assert np.all(np.abs(s - tau) >= 1e-3)          # generator keeps clear of tau
    expect = np.where(w.gate.built_below_tau, -1, w.gate.cand_prefix)
    assert m.tolist() == expect.tolist()
    if name == "tiny":
        assert m.tolist() == workloads.make_tiny_gate_tables()["map"]
        assert abs(s[0] - 1.0) < 1e-12 and 0.97 < s[1] < 0.99
