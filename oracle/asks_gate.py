"""ASKS similarity gate, fp64 (Eq. 2; Algorithm 2).

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np


def layer_weights(alpha: float, L: int) -> np.ndarray:
    """w_l = exp(alpha*l/L) / sum_l' exp(alpha*l'/L), l = 1..L  (text under Eq. 2; Alg. 2 line 1)."""
    l = np.arange(1, L + 1, dtype=np.float64)
    e = np.exp(np.float64(alpha) * l / np.float64(L))
    return e / e.sum()


def layer_cosines(h_b: np.ndarray, h_r: np.ndarray) -> np.ndarray:
    """cos(h_b^(l), h_root^(l)) for every layer l (the fraction inside Eq. 2).

    A zero-norm vector gives 0 for that layer (the paper does not say; this
    keeps the sum finite).
    """
    h_b = np.asarray(h_b, dtype=np.float64)
    h_r = np.asarray(h_r, dtype=np.float64)
    L = h_b.shape[0]
    c = np.zeros(L, dtype=np.float64)
    for l in range(L):
        dot = float(np.dot(h_b[l], h_r[l]))
        nb = float(np.dot(h_b[l], h_b[l]))
        nr = float(np.dot(h_r[l], h_r[l]))
        if nb > 0.0 and nr > 0.0:
            c[l] = dot / (np.sqrt(nb) * np.sqrt(nr))
        elif nb != nb or nr != nr:   # NaN input propagates
            c[l] = np.nan
    return c


def asks_gate(h_branch, h_root, cand_prefix, alpha: float, tau: float):
    """Branch-to-prefix map and similarities.

    h_branch [B][L][D], h_root [P][L][D] (raw or unit-norm: the norm is always
    divided out), cand_prefix [B] names the root each branch is compared with.
    sigma_b = sum_l w_l * cos_l (Eq. 2); map[b] = cand_prefix[b] if
    sigma_b >= tau else -1 (Alg. 2 lines 6-8: ">=").  alpha and tau are taken at
    fp32 precision, the precision in which the library receives them.
    """
    hb = np.asarray(h_branch, dtype=np.float64)
    hr = np.asarray(h_root, dtype=np.float64)
    cand = np.asarray(cand_prefix, dtype=np.int64)
    B, L, _ = hb.shape
    a = float(np.float32(alpha))
    t = float(np.float32(tau))
    w = layer_weights(a, L)
    sigma = np.zeros(B, dtype=np.float64)
    out = np.full(B, -1, dtype=np.int32)
    for b in range(B):
        r = int(cand[b])
        c = layer_cosines(hb[b], hr[r])
        s = 0.0
        for l in range(L):
            s += w[l] * c[l]
        sigma[b] = s
        if s >= t:
            out[b] = r
    return out, sigma
