"""Block tables that stand in for the paper's broadcast copy of the prefix cache.

Algorithm 1 line 3 makes B physical copies of the root cache; here a branch
that passed the gate simply lists the shared prefix's pages, and a branch that
failed it ("independent recomputation", Section 2.2) lists its own private
prefix pages.  Integer work only.  Test infrastructure: see the package docstring.
"""
from __future__ import annotations

import numpy as np


def tables_from_gate(branch_to_prefix, num_prefixes,
                     shared_off, shared_pages, shared_ntok,
                     priv_off, priv_pages, priv_ntok,
                     sfx_off, sfx_pages, sfx_ntok):
    """Segment tables from a gate map, in canonical order.

    Segments are numbered: shared prefixes by ascending prefix id (only those
    with at least one sharer), then the private prefix of every branch whose map
    entry is -1 by ascending branch (even if that list is empty), then every
    branch's suffix by ascending branch.  Branch b lists
    [its prefix segment, its suffix segment].
    Returns a dict of int32 arrays: seg_block_off, seg_blocks, seg_num_tokens,
    br_seg_off, br_segs.
    """
    m = np.asarray(branch_to_prefix, dtype=np.int64)
    B = m.shape[0]
    seg_pages = []
    seg_ntok = []
    shared_seg = {}
    for r in range(int(num_prefixes)):
        if np.any(m == r):
            shared_seg[r] = len(seg_pages)
            seg_pages.append(list(shared_pages[shared_off[r]:shared_off[r + 1]]))
            seg_ntok.append(int(shared_ntok[r]))
    priv_seg = {}
    for b in range(B):
        if m[b] < 0:
            priv_seg[b] = len(seg_pages)
            seg_pages.append(list(priv_pages[priv_off[b]:priv_off[b + 1]]))
            seg_ntok.append(int(priv_ntok[b]))
    sfx_seg = {}
    for b in range(B):
        sfx_seg[b] = len(seg_pages)
        seg_pages.append(list(sfx_pages[sfx_off[b]:sfx_off[b + 1]]))
        seg_ntok.append(int(sfx_ntok[b]))
    br_segs = []
    for b in range(B):
        first = shared_seg[int(m[b])] if m[b] >= 0 else priv_seg[b]
        br_segs += [first, sfx_seg[b]]
    seg_block_off = np.zeros(len(seg_pages) + 1, dtype=np.int32)
    seg_block_off[1:] = np.cumsum([len(p) for p in seg_pages])
    return {
        "seg_block_off": seg_block_off,
        "seg_blocks": np.array([p for pages in seg_pages for p in pages], dtype=np.int32),
        "seg_num_tokens": np.array(seg_ntok, dtype=np.int32),
        "br_seg_off": np.arange(0, 2 * B + 1, 2, dtype=np.int32),
        "br_segs": np.array(br_segs, dtype=np.int32),
    }


def segment_sharers(br_seg_off, br_segs, num_segments):
    """For every segment, the ascending list of branches that attend to it."""
    sharers = [[] for _ in range(int(num_segments))]
    B = len(br_seg_off) - 1
    for b in range(B):
        for s in br_segs[br_seg_off[b]:br_seg_off[b + 1]]:
            sharers[int(s)].append(b)
    return sharers


def logical_block_counts(seg_block_off, br_seg_off, br_segs):
    """Number of logical KV blocks of each branch (pages of its segments, concatenated)."""
    B = len(br_seg_off) - 1
    n = np.zeros(B, dtype=np.int64)
    for b in range(B):
        for s in br_segs[br_seg_off[b]:br_seg_off[b + 1]]:
            n[b] += int(seg_block_off[int(s) + 1]) - int(seg_block_off[int(s)])
    return n


def mass_offsets(seg_block_off, br_seg_off, br_segs):
    """Prefix sums of the logical block counts: branch b's masses start at off[b]*Hq."""
    n = logical_block_counts(seg_block_off, br_seg_off, br_segs)
    off = np.zeros(n.shape[0] + 1, dtype=np.int64)
    off[1:] = np.cumsum(n)
    return off
