"""One step of the token-by-token decode on the paged cache (Appendix "Stepwise Batched Decode",
step 2): where the new token's key and value go, and the tables afterwards.  Index work, exact.

Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np

BLOCK = 16


def append_token(seg_block_off, seg_blocks, seg_num_tokens, br_seg_off, br_segs, new_pages):
    """Every branch that lists segments gains one token at the end of its last segment.

    The last segment of a branch must be listed by that branch alone (its private suffix).  If that
    segment's pages are full (or it has none), page new_pages[b] is appended to it first.
    Returns (tables dict, page [B], slot [B]): where branch b's new token is stored (-1, -1 for a
    branch without segments).
    """
    S = len(seg_num_tokens)
    B = len(br_seg_off) - 1
    refs = np.zeros(S, dtype=np.int64)
    for s in br_segs:
        refs[int(s)] += 1
    pages = [[int(x) for x in seg_blocks[seg_block_off[s]:seg_block_off[s + 1]]] for s in range(S)]
    ntok = [int(x) for x in seg_num_tokens]
    page = np.full(B, -1, dtype=np.int32)
    slot = np.full(B, -1, dtype=np.int32)
    for b in range(B):
        if br_seg_off[b + 1] == br_seg_off[b]:
            continue
        s = int(br_segs[br_seg_off[b + 1] - 1])
        if refs[s] != 1:
            raise ValueError(f"the last segment of branch {b} is listed {refs[s]} times")
        if ntok[s] == len(pages[s]) * BLOCK:
            pages[s].append(int(new_pages[b]))
        page[b] = pages[s][-1]
        slot[b] = ntok[s] % BLOCK
        ntok[s] += 1
    off = np.zeros(S + 1, dtype=np.int32)
    for s in range(S):
        off[s + 1] = off[s] + len(pages[s])
    flat = np.asarray([p for ps in pages for p in ps], dtype=np.int32)
    t = {"seg_block_off": off, "seg_blocks": flat, "seg_num_tokens": np.asarray(ntok, dtype=np.int32),
         "br_seg_off": np.asarray(br_seg_off, dtype=np.int32), "br_segs": np.asarray(br_segs, dtype=np.int32)}
    return t, page, slot


def write_token(k_pool, v_pool, page, slot, k_new, v_new):
    """k_pool[page[b], :, slot[b], :] = k_new[b] (and v likewise) for every branch with page[b] >= 0.
    Pools [nblk][Hkv][16][d], k_new / v_new [B][Hkv][d]; in place."""
    for b in range(len(page)):
        if page[b] >= 0:
            k_pool[int(page[b]), :, int(slot[b]), :] = k_new[b]
            v_pool[int(page[b]), :, int(slot[b]), :] = v_new[b]
