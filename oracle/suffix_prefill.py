"""Suffix-prefill attention on the shared cache, fp64 (Section 2.2 "KV broadcast and batched
decode": y_b = f(s_b | C_B); Appendix "Stepwise Batched Decode", step (1): suffix prefill).

Test infrastructure: see the package docstring.

The s tokens of a branch's suffix are run through the model in one pass on top of the shared prefix
cache: query token i of branch b stands at position T_b - s + i of the branch's token sequence (the
keys and values of the s tokens are the last s tokens the branch's tables list) and attends to
every position up to and including its own - the whole prefix, whatever precedes the s tokens in
the branch's own segments, and the s tokens causally.
"""
from __future__ import annotations

import numpy as np

from .branch_attention import BLOCK, _gather_branch


def suffix_prefill_attention(num_q_heads, num_kv_heads, head_dim, sm_scale,
                             seg_block_off, seg_blocks, seg_num_tokens, br_seg_off, br_segs,
                             q, k_pool, v_pool, branches=None):
    """out[b][i][h] = softmax(scale * q[b][i][h] . K_b[:T_b - s + i + 1]^T) V_b[:T_b - s + i + 1].

    q [B][s][Hq][d]; everything else as in branch_decode_attention.  Returns (out [B][s][Hq][d] fp64,
    list over branches of mass [s][Hq][nblk_b] fp64: the softmax mass query token i of head h puts on
    the branch's j-th logical block).  A branch without tokens gets out = 0; one with some but
    fewer than s tokens is an error.
    """
    q = np.asarray(q, dtype=np.float64)
    B, s = q.shape[0], q.shape[1]
    G = num_q_heads // num_kv_heads
    scale = float(np.float32(sm_scale)) if sm_scale > 0 else 1.0 / np.sqrt(np.float64(head_dim))
    out = np.zeros((B, s, num_q_heads, head_dim), dtype=np.float64)
    masses = [None] * B
    for b in (range(B) if branches is None else branches):
        Kd, Vd, blk, nblk_b = _gather_branch(b, seg_block_off, seg_blocks, seg_num_tokens,
                                             br_seg_off, br_segs, k_pool, v_pool)
        T = 0 if Kd is None else Kd.shape[1]
        mass = np.zeros((s, num_q_heads, nblk_b), dtype=np.float64)
        masses[b] = mass
        if T == 0:
            continue                                  # a branch without tokens: out = 0, no masses
        if T < s:
            raise ValueError(f"branch {b} lists {T} tokens, fewer than the {s} suffix tokens")
        for i in range(s):
            Tv = T - s + i + 1                       # positions 0 .. T - s + i
            for h in range(num_q_heads):
                g = h // G
                sc = scale * (Kd[g, :Tv] @ q[b, i, h])
                e = np.exp(sc - sc.max())
                p = e / e.sum()
                out[b, i, h] = p @ Vd[g, :Tv]
                mass[i, h] = np.bincount(blk[:Tv], weights=p, minlength=nblk_b)
    return out, masses


def suffix_prefill_tables(seg_block_off, seg_blocks, seg_num_tokens, br_seg_off, br_segs, s):
    """Tables that turn the suffix prefill into a decode attention over B * s virtual branches.

    Virtual branch b * s + i is query token i of branch b.  It lists every segment of b but the
    last unchanged, then two new segments cut from b's last segment: its pages that lie wholly
    before the first of the s tokens (shared by the s virtual branches of b, possibly empty), and
    the pages from there up to the one holding query token i, with only the tokens up to token i's
    own counted.  New
    segments are numbered after the original ones, branch by branch: the common part of b is
    segment S + b * (s + 1), the part of token i is S + b * (s + 1) + 1 + i.  The last segment of a
    branch must hold at least s tokens.  A branch without segments yields s empty virtual branches.
    The logical blocks of a virtual branch are the leading blocks of the branch, in the same order
    (blocks that hold only later tokens are not listed).
    Returns a dict of int32 arrays with the five table fields.
    """
    S = len(seg_num_tokens)
    B = len(br_seg_off) - 1
    off = [int(x) for x in seg_block_off]
    blocks = [int(x) for x in seg_blocks]
    ntok = [int(x) for x in seg_num_tokens]
    new_br_off, new_br_segs = [0], []
    for b in range(B):
        segs = [int(x) for x in br_segs[br_seg_off[b]:br_seg_off[b + 1]]]
        if not segs:
            for i in range(s + 1):                    # keep the numbering uniform: s + 1 empty segments
                off.append(len(blocks))
                ntok.append(0)
            for i in range(s):
                new_br_off.append(len(new_br_segs))
            continue
        last = segs[-1]
        lo, hi, T = int(seg_block_off[last]), int(seg_block_off[last + 1]), int(seg_num_tokens[last])
        if T < s:
            raise ValueError(f"the last segment of branch {b} holds {T} tokens, fewer than {s}")
        ncommon = (T - s) // BLOCK                    # pages wholly before the first suffix token
        blocks.extend(int(x) for x in seg_blocks[lo:lo + ncommon])
        off.append(len(blocks))
        ntok.append(ncommon * BLOCK)
        for i in range(s):
            nt = T - s + i + 1 - ncommon * BLOCK      # tokens of the tail part that token i sees (>= 1)
            npg = (nt + BLOCK - 1) // BLOCK
            blocks.extend(int(x) for x in seg_blocks[lo + ncommon:lo + ncommon + npg])
            off.append(len(blocks))
            ntok.append(nt)
        for i in range(s):
            new_br_segs.extend(segs[:-1] + [S + b * (s + 1), S + b * (s + 1) + 1 + i])
            new_br_off.append(len(new_br_segs))
    a = lambda v: np.asarray(v, dtype=np.int32)
    return {"seg_block_off": a(off), "seg_blocks": a(blocks), "seg_num_tokens": a(ntok),
            "br_seg_off": a(new_br_off), "br_segs": a(new_br_segs)}
