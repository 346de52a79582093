"""CGEE numerics, fp64 (Section 2.3: Eq. 3-5; Algorithm 3).

Test infrastructure: see the package docstring.

* ``logit_entropy``: H = -sum_v p_v log p_v with p = softmax(h W_u^T) (Eq. 5), per row of h, in
  nats, and the top-1 probability max_v p_v of the same distribution (the summand of Eq. 3).
* ``entropy_exit``: the exit test of Algorithm 3 for layer l given H and the previous layer's H.
* ``generation_confidence``: Eq. 3, the mean top-1 probability over the decode steps.
* ``verify_skip``: the Level-1 gate of Eq. 4.
"""
from __future__ import annotations

import numpy as np


def logit_entropy(h, w_u):
    """h [B][D], w_u [V][D] (any float arrays; taken as fp64).  Returns (H [B] nats, top1 [B])."""
    h = np.asarray(h, dtype=np.float64)
    w = np.asarray(w_u, dtype=np.float64)
    z = h @ w.T                                        # [B][V]
    z = z - z.max(axis=1, keepdims=True)
    e = np.exp(z)
    p = e / e.sum(axis=1, keepdims=True)
    with np.errstate(divide="ignore", invalid="ignore"):
        plogp = np.where(p > 0, p * np.log(p), 0.0)
    return -plogp.sum(axis=1), p.max(axis=1)


def entropy_exit(H, H_prev, layer, l_min, theta, eps):
    """Algorithm 3's test, per row: layer >= l_min and H < theta and |H - H_prev| < eps.
    H_prev = +inf before the first layer, which makes the last condition false."""
    H = np.asarray(H, dtype=np.float64)
    H_prev = np.asarray(H_prev, dtype=np.float64)
    with np.errstate(invalid="ignore"):
        stable = np.abs(H - H_prev) < eps
    return (layer >= l_min) & (H < theta) & stable


def generation_confidence(top1_per_step):
    """Eq. 3: top1_per_step [t][B] -> p [B], the mean over the t decode steps."""
    return np.asarray(top1_per_step, dtype=np.float64).mean(axis=0)


def verify_skip(p, tau_conf, r_gap):
    """Eq. 4: max_b p >= tau_conf and (max - 2nd max) / max >= r_gap.  With one branch there is no
    competitor: the second maximum is taken as 0 (gap 1)."""
    p = np.asarray(p, dtype=np.float64)
    if p.size == 0:
        return False
    srt = np.sort(p)[::-1]
    top = srt[0]
    second = srt[1] if p.size > 1 else 0.0
    if not top > 0:
        return False
    return bool(top >= tau_conf and (top - second) / top >= r_gap)
