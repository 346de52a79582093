"""RSBCM: attention-weighted, depth-discounted block eviction, fp64 (Section 2.4; Algorithm 4).

Test infrastructure: see the package docstring.

The paper scores a cached block by omega = score / (depth + 1) and, while more than N_max blocks
are cached, evicts the block with the smallest omega.  It does not define an attention-derived
score; the reading taken here is: the score of a table entry (a page of a segment) is the softmax
mass that every (branch, query head) attending to the segment puts on that page, summed.
"""
from __future__ import annotations

import numpy as np


def page_scores(seg_block_off, br_seg_off, br_segs, masses, num_q_heads):
    """score[e] for every table entry e = seg_block_off[s] + p (page p of segment s).

    masses[b] is [Hq][nblk_b] (fp32 or fp64), logical block j of branch b being the j-th page of the
    concatenation of its segments.  score[e] = sum over the branches b listing s (ascending b; a
    branch listing s twice counts twice) of [ sum over heads h (ascending) of masses[b][h][j] ]:
    the head sum of a branch is formed first, then added to the running score, all in fp64 and in
    exactly that order, so that another implementation can reproduce the value bit for bit.
    """
    S = len(seg_block_off) - 1
    score = np.zeros(int(seg_block_off[S]), dtype=np.float64)
    B = len(br_seg_off) - 1
    for b in range(B):
        loff = 0
        m = np.asarray(masses[b], dtype=np.float64)
        for s in br_segs[br_seg_off[b]:br_seg_off[b + 1]]:
            s = int(s)
            lo, hi = int(seg_block_off[s]), int(seg_block_off[s + 1])
            head_sum = np.zeros(hi - lo, dtype=np.float64)
            for h in range(int(num_q_heads)):
                head_sum += m[h, loff:loff + (hi - lo)]
            score[lo:hi] += head_sum
            loff += hi - lo
    return score


def apply_eviction(seg_block_off, seg_blocks, seg_num_tokens, evicted, block_size=16):
    """Tables after the evicted entries are dropped: each segment keeps its surviving pages in
    order; a dropped page takes its tokens with it (every page of a segment holds block_size
    tokens except the last, which holds the remainder).  Branch lists are unchanged.
    Returns (seg_block_off, seg_blocks, seg_num_tokens) as int32 arrays.
    """
    S = len(seg_block_off) - 1
    new_off, new_blocks, new_ntok = [0], [], []
    for s in range(S):
        lo, hi = int(seg_block_off[s]), int(seg_block_off[s + 1])
        ntok = int(seg_num_tokens[s])
        kept_tokens = 0
        for p in range(hi - lo):
            in_page = min(block_size, ntok - p * block_size)
            if not evicted[lo + p]:
                new_blocks.append(int(seg_blocks[lo + p]))
                kept_tokens += in_page
        new_off.append(len(new_blocks))
        new_ntok.append(kept_tokens)
    return (np.asarray(new_off, np.int32), np.asarray(new_blocks, np.int32), np.asarray(new_ntok, np.int32))


def rsbcm_evict(score, depth, capacity):
    """Algorithm 4, literally: while more than `capacity` entries remain, recompute omega for the
    remaining ones and evict the arg-min (the first one, if several share the minimum).

    score fp64 [N], depth int [N].  Returns (evicted bool [N], order: entry indices in eviction order).
    """
    score = np.asarray(score, dtype=np.float64)
    depth = np.asarray(depth, dtype=np.int64)
    alive = list(range(score.shape[0]))
    order = []
    while len(alive) > capacity:
        omega = [score[i] / np.float64(depth[i] + 1) for i in alive]
        k = int(np.argmin(np.asarray(omega, dtype=np.float64)))
        order.append(alive.pop(k))
    evicted = np.zeros(score.shape[0], dtype=bool)
    evicted[order] = True
    return evicted, np.asarray(order, dtype=np.int64)
