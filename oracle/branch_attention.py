"""Decode attention of every branch over a physically duplicated prefix + suffix, fp64.

This is the plain definition the shared-prefix kernels must reproduce: sharing
changes where the bytes come from, not the value.  Each branch gets its own
contiguous copy of all the KV it attends to (what the paper builds with
repeat_interleave + clone, Section 2.2), then ordinary softmax attention with
one query per (branch, head).  Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

BLOCK = 16


def to_f32_numpy(x) -> np.ndarray:
    """A torch tensor (any float dtype, bf16 included) or array as an fp32 numpy array (exact for bf16)."""
    if hasattr(x, "detach"):
        x = x.detach().cpu().float().numpy()
    return np.asarray(x, dtype=np.float32)


def _gather_branch(b, seg_block_off, seg_blocks, seg_num_tokens, br_seg_off, br_segs,
                   k_pool, v_pool):
    """Copy the valid tokens of every page branch b lists, in order.

    Returns Kd, Vd as [Hkv][T_b][d] fp64, the logical block index of every
    token, and the number of logical blocks.
    """
    ks, vs, blk = [], [], []
    j = 0
    for s in br_segs[br_seg_off[b]:br_seg_off[b + 1]]:
        s = int(s)
        pages = seg_blocks[seg_block_off[s]:seg_block_off[s + 1]]
        ntok = int(seg_num_tokens[s])
        for i, page in enumerate(pages):
            valid = min(BLOCK, ntok - BLOCK * i)
            if valid > 0:
                ks.append(np.asarray(k_pool[int(page), :, :valid, :], dtype=np.float64))
                vs.append(np.asarray(v_pool[int(page), :, :valid, :], dtype=np.float64))
                blk.append(np.full(valid, j, dtype=np.int64))
            j += 1
    if not ks:
        return None, None, np.zeros(0, dtype=np.int64), j
    return (np.concatenate(ks, axis=1), np.concatenate(vs, axis=1), np.concatenate(blk), j)


def branch_decode_attention(num_q_heads, num_kv_heads, head_dim, sm_scale,
                            seg_block_off, seg_blocks, seg_num_tokens, br_seg_off, br_segs,
                            q, k_pool, v_pool, branches=None):
    """out[b][h] = softmax(scale * q[b][h] . K_b^T) V_b and the softmax mass per logical block.

    q [B][Hq][d]; pools [nblk][Hkv][16][d] (fp32 arrays holding bf16 values);
    q-head h reads kv-head h // (Hq/Hkv).  scale = sm_scale if > 0 else
    1/sqrt(d).  No mask: the decode query attends to every listed token.  A
    branch with no tokens gets out = 0 and no masses.
    Returns (out [B][Hq][d] fp64, list over branches of mass [Hq][nblk_b] fp64).
    ``branches`` restricts the work to a subset (other rows stay 0 / None).
    """
    q = np.asarray(q, dtype=np.float64)
    B = q.shape[0]
    G = num_q_heads // num_kv_heads
    scale = float(np.float32(sm_scale)) if sm_scale > 0 else 1.0 / np.sqrt(np.float64(head_dim))
    out = np.zeros((B, num_q_heads, head_dim), dtype=np.float64)
    masses = [None] * B
    todo = range(B) if branches is None else branches
    for b in todo:
        Kd, Vd, blk, nblk_b = _gather_branch(b, seg_block_off, seg_blocks, seg_num_tokens,
                                             br_seg_off, br_segs, k_pool, v_pool)
        mass = np.zeros((num_q_heads, nblk_b), dtype=np.float64)
        masses[b] = mass
        if Kd is None:
            continue
        for h in range(num_q_heads):
            g = h // G
            s = scale * (Kd[g] @ q[b, h])
            m = s.max()
            e = np.exp(s - m)
            p = e / e.sum()
            out[b, h] = p @ Vd[g]
            mass[h] = np.bincount(blk, weights=p, minlength=nblk_b)
    return out, masses
