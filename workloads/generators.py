"""Seeded synthetic inputs shaped like the paper's workloads.

What the shapes stand for (the paper's benchmark items are not used anywhere):
B = 8 branches per problem, prefix about 1024 tokens, short per-branch suffixes
(Section 3.1 and the hyper-parameter table of Appendix C), the head layouts of
the 7B-10B models it evaluates (Section 3.1), and a Tree-of-Thoughts tree with
branching 4 and depth 3 (Section 1).  All values are N(0,1): Q/K/V are drawn in
fp32 and rounded to bf16 (round to nearest even, by torch); hidden states stay
fp32.

Conventions shared by every workload:

* KV pool layout ``[num_pool_blocks][num_kv_heads][16][head_dim]`` bf16, K and
  V in separate tensors.  A *page* (block) holds 16 tokens of every KV head.
* A *segment* is an ordered list of physical pages plus a token count; only its
  last page may be partial.  A branch's KV is the concatenation of its segments
  in root-to-leaf order.
* K/V values are drawn in logical order (data segment, page, kv head, token,
  dim) and then scattered to physical pages through a seeded permutation, so
  what a branch sees does not depend on the permutation.
* Slots past a segment's token count, and pages nobody references, hold a large
  finite sentinel so that a reader that ignores the token count is far off
  (never NaN/Inf).

Nothing here computes a similarity, a softmax or a table from a gate map.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import numpy as np
import torch

BLOCK = 16
SENTINEL = 1.0e4
SEED_BASE = 42  # the paper fixes seed 42 for its runs (Section 3.1)

CONFIG_NAMES = ("tiny", "qwen_layer", "tot", "batched_serving", "long_context")


@dataclasses.dataclass
class Layout:
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    num_pool_blocks: int
    block_size: int = BLOCK
    sm_scale: float = 0.0  # <= 0 means 1/sqrt(head_dim)

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def bytes_per_token(self) -> int:
        return 2 * self.num_kv_heads * self.head_dim * 2


@dataclasses.dataclass
class Tables:
    """Segment form of the block tables (all int32 numpy arrays)."""
    seg_block_off: np.ndarray   # [S+1]
    seg_blocks: np.ndarray      # physical page ids, segment-major
    seg_num_tokens: np.ndarray  # [S]
    br_seg_off: np.ndarray      # [B+1]
    br_segs: np.ndarray         # segment ids, root-to-leaf per branch

    @property
    def num_segments(self) -> int:
        return int(self.seg_num_tokens.shape[0])

    @property
    def num_branches(self) -> int:
        return int(self.br_seg_off.shape[0]) - 1


@dataclasses.dataclass
class FlatLists:
    """Two-level form: P shared prefixes, per-branch private prefix copy and suffix."""
    num_prefixes: int
    shared_off: np.ndarray
    shared_pages: np.ndarray
    shared_ntok: np.ndarray
    priv_off: np.ndarray
    priv_pages: np.ndarray
    priv_ntok: np.ndarray
    sfx_off: np.ndarray
    sfx_pages: np.ndarray
    sfx_ntok: np.ndarray


@dataclasses.dataclass
class GateInputs:
    h_branch: torch.Tensor     # [B][L][D] fp32
    h_root: torch.Tensor       # [P][L][D] fp32
    cand_prefix: np.ndarray    # [B] int32
    alpha: float
    tau: float
    built_below_tau: np.ndarray  # [B] bool: branches drawn far from their root


@dataclasses.dataclass
class Workload:
    name: str
    layout: Layout
    q: torch.Tensor            # [B][Hq][d] bf16
    k_pool: torch.Tensor       # [nblk][Hkv][16][d] bf16
    v_pool: torch.Tensor
    tables: Optional[Tables] = None   # given tables, when the config states them
    flat: Optional[FlatLists] = None  # two-level lists, when tables come from the gate
    gate: Optional[GateInputs] = None
    notes: str = ""
    phrasing_level: Optional[np.ndarray] = None   # diverse-phrasing regime: divergence level of each branch

    @property
    def num_branches(self) -> int:
        return int(self.q.shape[0])


# --------------------------------------------------------------------------------------
# low-level drawing
# --------------------------------------------------------------------------------------

def _torch_gen(seed: int, tag: int) -> torch.Generator:
    g = torch.Generator(device="cpu")
    g.manual_seed((int(seed) * 1000003 + int(tag)) & 0x7FFFFFFFFFFFFFFF)
    return g


def _randn_bf16(shape, gen: torch.Generator, chunk_rows: int = 2048) -> torch.Tensor:
    """N(0,1) in fp32, rounded to bf16; drawn chunk by chunk along dim 0 to bound memory."""
    out = torch.empty(shape, dtype=torch.bfloat16)
    n0 = shape[0]
    for lo in range(0, n0, chunk_rows):
        hi = min(n0, lo + chunk_rows)
        out[lo:hi] = torch.randn((hi - lo,) + tuple(shape[1:]), generator=gen,
                                 dtype=torch.float32).to(torch.bfloat16)
    return out


def _pages_of(ntok: int) -> int:
    return (int(ntok) + BLOCK - 1) // BLOCK


def _build_pool(seg_ntok: Sequence[int], num_kv_heads: int, head_dim: int, seed: int,
                spare_frac: float = 0.125):
    """Draw K/V for the given data segments and scatter them over a permuted pool.

    Returns (k_pool, v_pool, seg_block_off, seg_blocks, num_pool_blocks).
    """
    seg_ntok = [int(n) for n in seg_ntok]
    npages = [_pages_of(n) for n in seg_ntok]
    used = int(sum(npages))
    nblk = used + max(1, int(math.ceil(used * spare_frac)))
    rng = np.random.default_rng([SEED_BASE, int(seed), 7])
    perm = rng.permutation(nblk).astype(np.int32)
    seg_block_off = np.zeros(len(seg_ntok) + 1, dtype=np.int32)
    seg_block_off[1:] = np.cumsum(npages)
    seg_blocks = perm[:used].copy()

    shape = (used, num_kv_heads, BLOCK, head_dim)
    k_log = _randn_bf16(shape, _torch_gen(seed, 1))
    v_log = _randn_bf16(shape, _torch_gen(seed, 2))
    for s, n in enumerate(seg_ntok):
        r = n % BLOCK
        if n > 0 and r != 0:
            last = int(seg_block_off[s + 1]) - 1
            k_log[last, :, r:, :] = SENTINEL
            v_log[last, :, r:, :] = SENTINEL
    pool_shape = (nblk, num_kv_heads, BLOCK, head_dim)
    k_pool = torch.full(pool_shape, SENTINEL, dtype=torch.bfloat16)
    v_pool = torch.full(pool_shape, SENTINEL, dtype=torch.bfloat16)
    idx = torch.from_numpy(seg_blocks.astype(np.int64))
    k_pool[idx] = k_log
    v_pool[idx] = v_log
    return k_pool, v_pool, seg_block_off, seg_blocks, nblk


def _csr(lists: Sequence[Sequence[int]]):
    off = np.zeros(len(lists) + 1, dtype=np.int32)
    off[1:] = np.cumsum([len(x) for x in lists])
    flat = np.array([v for x in lists for v in x], dtype=np.int32)
    return off, flat


def make_gate_inputs(cand_prefix: Sequence[int], num_prefixes: int, L: int, D: int,
                     eps: Sequence[float], alpha: float, tau: float, seed: int,
                     root_from_branch0: bool = False) -> GateInputs:
    """Hidden states with a controlled angle to the candidate root.

    ``h_branch[b] = h_root[cand[b]] + eps[b] * noise_b`` per layer, all N(0,1) in
    fp32; ``eps[b] = inf`` draws the branch independently of its root.  With
    ``root_from_branch0`` the single root is a copy of branch 0 (the tiny
    config's "noisy copies of branch 0").
    """
    cand = np.asarray(cand_prefix, dtype=np.int32)
    B = cand.shape[0]
    g = _torch_gen(seed, 3)
    h_root = torch.randn((num_prefixes, L, D), generator=g, dtype=torch.float32)
    noise = torch.randn((B, L, D), generator=g, dtype=torch.float32)
    h_branch = torch.empty((B, L, D), dtype=torch.float32)
    eps = [float(e) for e in eps]
    for b in range(B):
        if math.isinf(eps[b]):
            h_branch[b] = noise[b]
        else:
            h_branch[b] = h_root[int(cand[b])] + eps[b] * noise[b]
    if root_from_branch0:
        assert num_prefixes == 1
        h_root = h_branch[0:1].clone()
    below = np.array([not (e < 0.5) for e in eps], dtype=bool)
    return GateInputs(h_branch=h_branch.contiguous(), h_root=h_root.contiguous(),
                      cand_prefix=cand, alpha=float(alpha), tau=float(tau),
                      built_below_tau=below)


# --------------------------------------------------------------------------------------
# generic builder used by the edge-case tests
# --------------------------------------------------------------------------------------

def make_from_segments(name: str, num_q_heads: int, num_kv_heads: int, head_dim: int,
                       seg_ntok: Sequence[int], br_segs: Sequence[Sequence[int]],
                       seed: int, sm_scale: float = 0.0, q_gain: float = 1.0) -> Workload:
    """A workload from explicit segment lengths and per-branch segment lists."""
    k_pool, v_pool, seg_block_off, seg_blocks, nblk = _build_pool(
        seg_ntok, num_kv_heads, head_dim, seed)
    B = len(br_segs)
    q = (_randn_bf16((max(B, 1), num_q_heads, head_dim), _torch_gen(seed, 4)).float()
         * q_gain).to(torch.bfloat16)[:B]
    br_off, br_flat = _csr(br_segs)
    tables = Tables(seg_block_off=seg_block_off, seg_blocks=seg_blocks,
                    seg_num_tokens=np.asarray(seg_ntok, dtype=np.int32),
                    br_seg_off=br_off, br_segs=br_flat)
    layout = Layout(num_q_heads, num_kv_heads, head_dim, nblk, sm_scale=sm_scale)
    return Workload(name=name, layout=layout, q=q, k_pool=k_pool, v_pool=v_pool, tables=tables)


def _two_level(name, num_q_heads, num_kv_heads, head_dim, prefix_ntok, branch_problem,
               priv_branches, sfx_ntok, seed) -> Workload:
    """P shared prefixes, private prefix copies for ``priv_branches``, one suffix per branch.

    Data segments in order: shared prefixes (ascending p), private copies
    (ascending b, same length as the branch's problem prefix, independent
    values), suffixes (ascending b).  ``tables`` references the shared prefix
    for every branch (the "as stated" reading); ``flat`` carries the lists from
    which gate-driven tables are built.
    """
    P = len(prefix_ntok)
    B = len(branch_problem)
    priv_set = sorted(int(b) for b in priv_branches)
    seg_ntok = list(int(n) for n in prefix_ntok)
    seg_ntok += [int(prefix_ntok[branch_problem[b]]) for b in priv_set]
    seg_ntok += list(int(n) for n in sfx_ntok)
    k_pool, v_pool, seg_block_off, seg_blocks, nblk = _build_pool(
        seg_ntok, num_kv_heads, head_dim, seed)

    def pages(s):
        return seg_blocks[seg_block_off[s]:seg_block_off[s + 1]].tolist()

    shared_lists = [pages(p) for p in range(P)]
    priv_lists = [[] for _ in range(B)]
    priv_ntok = np.zeros(B, dtype=np.int32)
    for i, b in enumerate(priv_set):
        priv_lists[b] = pages(P + i)
        priv_ntok[b] = seg_ntok[P + i]
    sfx_base = P + len(priv_set)
    sfx_lists = [pages(sfx_base + b) for b in range(B)]
    so, sp = _csr(shared_lists)
    po, pp = _csr(priv_lists)
    xo, xp = _csr(sfx_lists)
    flat = FlatLists(num_prefixes=P, shared_off=so, shared_pages=sp,
                     shared_ntok=np.asarray(prefix_ntok, dtype=np.int32),
                     priv_off=po, priv_pages=pp, priv_ntok=priv_ntok,
                     sfx_off=xo, sfx_pages=xp, sfx_ntok=np.asarray(sfx_ntok, dtype=np.int32))
    br_segs = [[int(branch_problem[b]), sfx_base + b] for b in range(B)]
    br_off, br_flat = _csr(br_segs)
    tables = Tables(seg_block_off=seg_block_off, seg_blocks=seg_blocks,
                    seg_num_tokens=np.asarray(seg_ntok, dtype=np.int32),
                    br_seg_off=br_off, br_segs=br_flat)
    q = _randn_bf16((B, num_q_heads, head_dim), _torch_gen(seed, 4))
    layout = Layout(num_q_heads, num_kv_heads, head_dim, nblk)
    return Workload(name=name, layout=layout, q=q, k_pool=k_pool, v_pool=v_pool,
                    tables=tables, flat=flat)


# --------------------------------------------------------------------------------------
# the five configurations
# --------------------------------------------------------------------------------------

EPS_NEAR = 0.203   # cos about 0.98
EPS_FAR = 0.75     # cos about 0.80


def make_tiny(seed: int = SEED_BASE + 0) -> Workload:
    """Config 1: 8 q / 2 kv heads, d 64, 4 branches on one 256-token prefix + 32-token suffixes.

    ``tables`` is the configuration as stated (all four branches share).  ``flat``
    and ``gate`` give the end-to-end variant: root = branch 0, branches 1-2 noisy
    copies, branch 3 independent (it has a private prefix copy).
    """
    w = _two_level("tiny", 8, 2, 64, [256], [0, 0, 0, 0], [3], [32, 32, 32, 32], seed)
    w.gate = make_gate_inputs([0, 0, 0, 0], 1, 4, 256, [0.0, EPS_NEAR, EPS_NEAR, math.inf],
                              alpha=0.5, tau=0.9, seed=seed, root_from_branch0=True)
    return w


def make_tiny_gate_tables():
    """Hand-written expected result of config 1's end-to-end variant (map, segment lists)."""
    return {"map": [0, 0, 0, -1],
            # segments: shared prefix 0; private prefix of branch 3; suffixes 0..3
            "br_segs": [[0, 2], [0, 3], [0, 4], [1, 5]],
            "seg_num_tokens": [256, 256, 32, 32, 32, 32]}


def make_qwen_layer(seed: int = SEED_BASE + 1, prefix: int = 2048, suffix: int = 512) -> Workload:
    """Config 2: 28 q / 4 kv heads, d 128, 4 branches, prefix 2048, suffix 512; gate [4,28,3584]."""
    w = _two_level("qwen_layer", 28, 4, 128, [prefix], [0] * 4, [], [suffix] * 4, seed)
    w.gate = make_gate_inputs([0] * 4, 1, 28, 3584, [EPS_NEAR] * 4, alpha=0.5, tau=0.9, seed=seed)
    return w


def make_tot(seed: int = SEED_BASE + 2, branching: int = 4, depth: int = 3,
             root_tokens: int = 1024, level_tokens: int = 256,
             num_q_heads: int = 32, num_kv_heads: int = 8, head_dim: int = 128) -> Workload:
    """Config 3: Tree-of-Thoughts tree, one segment per node in BFS order, leaves are branches."""
    seg_ntok = [root_tokens]
    level_start = [0]
    for lev in range(1, depth + 1):
        level_start.append(len(seg_ntok))
        seg_ntok += [level_tokens] * (branching ** lev)
    num_leaves = branching ** depth
    br_segs = []
    for leaf in range(num_leaves):
        path = [0]
        for lev in range(1, depth + 1):
            path.append(level_start[lev] + leaf // (branching ** (depth - lev)))
        br_segs.append(path)
    w = make_from_segments("tot", num_q_heads, num_kv_heads, head_dim, seg_ntok, br_segs, seed)
    w.notes = f"ToT branching {branching} depth {depth}: {len(seg_ntok)} node segments"
    return w


def make_batched_serving(seed: int = SEED_BASE + 3, problems: int = 32, branches_per: int = 8,
                         prefix_range=(512, 4096), suffix_range=(128, 1024),
                         perturbed_frac: float = 0.3, L: int = 28, D: int = 3584,
                         num_q_heads: int = 28, num_kv_heads: int = 4,
                         head_dim: int = 128) -> Workload:
    """Config 4: problems x branches, uniform prefix/suffix lengths, 30% of branches built below tau."""
    rng = np.random.default_rng([SEED_BASE, int(seed), 11])
    B = problems * branches_per
    prefix_ntok = rng.integers(prefix_range[0], prefix_range[1], size=problems, endpoint=True)
    sfx_ntok = rng.integers(suffix_range[0], suffix_range[1], size=B, endpoint=True)
    n_pert = int(round(perturbed_frac * B))
    pert = np.sort(rng.choice(B, size=n_pert, replace=False))
    branch_problem = [b // branches_per for b in range(B)]
    w = _two_level("batched_serving", num_q_heads, num_kv_heads, head_dim, prefix_ntok.tolist(),
                   branch_problem, pert.tolist(), sfx_ntok.tolist(), seed)
    eps = [EPS_NEAR] * B
    for b in pert:
        eps[int(b)] = EPS_FAR
    w.gate = make_gate_inputs(branch_problem, problems, L, D, eps, alpha=0.5, tau=0.9, seed=seed)
    w.tables = None  # this config is end to end: tables come from the gate map
    w.notes = f"{problems} problems x {branches_per} branches, {n_pert} branches built below tau"
    return w


def make_long_context(seed: int = SEED_BASE + 4, prefix: int = 32768, suffix: int = 2048,
                      branches: int = 16, num_q_heads: int = 32, num_kv_heads: int = 8,
                      head_dim: int = 128) -> Workload:
    """Config 5 before eviction: one long shared prefix + per-branch suffixes (full tables).

    ``punch_holes`` removes the evicted pages from the prefix segment.
    """
    w = _two_level("long_context", num_q_heads, num_kv_heads, head_dim, [prefix], [0] * branches,
                   [], [suffix] * branches, seed)
    w.notes = "full tables; holes are punched by punch_holes()"
    return w


# eps of the four semantic-divergence levels of the diverse-phrasing regime (cos = 1 / sqrt(1 + eps^2)):
# identical 1.0, minor rewording 0.94, structural reframing 0.74, very different register 0.45
PHRASING_EPS = (0.0, 0.35, 0.9, 2.0)


def make_diverse_phrasing(seed: int = SEED_BASE + 5, problems: int = 15, templates: int = 8,
                          prefix: int = 512, sfx_lo: int = 16, sfx_hi: int = 144,
                          num_q_heads: int = 28, num_kv_heads: int = 4, head_dim: int = 128,
                          L: int = 28, D: int = 3584) -> Workload:
    """The diverse-phrasing regime of Section "ASKS Novelty Over vLLM Prefix Caching": every problem is
    posed through ``templates`` phrasings spread evenly over four semantic-divergence levels, padded to
    about ``prefix`` tokens; phrasing 0 is the problem's root.  Qwen2.5-7B shapes, the paper's default
    alpha = 1.5 and tau = 0.82.  The hidden states of a phrasing sit at the angle of its level from the
    root's (PHRASING_EPS), so the two closer levels pass the gate and the two farther ones keep a
    private prefix.  Tables come from the gate map (end to end, like the batched-serving config).

    ``w.notes`` records which branches an exact-token prefix cache could share (level 0 only)."""
    assert templates % 4 == 0
    per_level = templates // 4
    B = problems * templates
    rng = np.random.default_rng([SEED_BASE, int(seed), 13])
    level = np.array([(b % templates) // per_level for b in range(B)], dtype=np.int32)
    branch_problem = [b // templates for b in range(B)]
    sfx_ntok = rng.integers(sfx_lo, sfx_hi + 1, size=B)
    far = np.flatnonzero(level >= 2)
    w = _two_level("diverse_phrasing", num_q_heads, num_kv_heads, head_dim, [prefix] * problems,
                   branch_problem, far.tolist(), sfx_ntok.tolist(), seed)
    eps = [PHRASING_EPS[int(l)] for l in level]
    w.gate = make_gate_inputs(branch_problem, problems, L, D, eps, alpha=1.5, tau=0.82, seed=seed)
    w.tables = None
    w.phrasing_level = level
    w.notes = (f"{problems} problems x {templates} phrasings at 4 divergence levels; an exact-token cache "
               f"shares level 0 only, the gate is built to share levels 0 and 1")
    return w


def lowest_mass_pages(scores: np.ndarray, frac: float = 0.2) -> np.ndarray:
    """Logical indices of the floor(frac*n) pages with the lowest score (ties: lower index)."""
    scores = np.asarray(scores, dtype=np.float64)
    n = scores.shape[0]
    k = int(math.floor(frac * n))
    order = np.argsort(scores, kind="stable")
    return np.sort(order[:k]).astype(np.int64)


def punch_holes(w: Workload, segment: int, evicted_logical_pages: np.ndarray) -> Workload:
    """A copy of ``w`` whose tables no longer list the given pages of ``segment``.

    Pages are only removed from the table (the pool is untouched).  The
    segment's token count drops by 16 per removed full page; the last page may
    be removed too, in which case the new last page is a full one.
    """
    t = w.tables
    lo, hi = int(t.seg_block_off[segment]), int(t.seg_block_off[segment + 1])
    npg = hi - lo
    ntok = int(t.seg_num_tokens[segment])
    keep = np.ones(npg, dtype=bool)
    keep[np.asarray(evicted_logical_pages, dtype=np.int64)] = False
    valid = np.full(npg, BLOCK, dtype=np.int64)
    if npg > 0:
        valid[-1] = ntok - (npg - 1) * BLOCK
    new_ntok = int(valid[keep].sum())
    kept_pages = t.seg_blocks[lo:hi][keep]
    seg_blocks = np.concatenate([t.seg_blocks[:lo], kept_pages, t.seg_blocks[hi:]]).astype(np.int32)
    seg_block_off = t.seg_block_off.copy()
    seg_block_off[segment + 1:] -= (npg - int(keep.sum()))
    seg_num_tokens = t.seg_num_tokens.copy()
    seg_num_tokens[segment] = new_ntok
    nt = Tables(seg_block_off=seg_block_off, seg_blocks=seg_blocks, seg_num_tokens=seg_num_tokens,
                br_seg_off=t.br_seg_off.copy(), br_segs=t.br_segs.copy())
    out = dataclasses.replace(w, tables=nt, flat=None)
    out.name = w.name + "+holes"
    return out


def make_block_masses(t: Tables, num_q_heads: int, seed: int = SEED_BASE + 50) -> list:
    """Synthetic stand-ins for the attention's second output: for every branch an fp32 array
    [Hq][nblk_b] of non-negative numbers, each row scaled to sum to about 1, with the heavy
    tail real softmax masses have (a few blocks take most of the mass, many are near zero)."""
    rng = np.random.default_rng(seed)
    out = []
    for b in range(t.num_branches):
        segs = t.br_segs[t.br_seg_off[b]:t.br_seg_off[b + 1]]
        nblk = int(sum(int(t.seg_block_off[s + 1] - t.seg_block_off[s]) for s in segs))
        m = np.exp(4.0 * rng.standard_normal((num_q_heads, nblk)))
        m /= np.maximum(m.sum(axis=1, keepdims=True), 1e-300)
        out.append(m.astype(np.float32))
    return out


def make_eviction_inputs(n: int, seed: int = SEED_BASE + 51, max_depth: int = 6, tie_levels: int = 0):
    """(score fp64 [n] >= 0, depth int32 [n]) for an eviction.  tie_levels > 0 draws the scores from
    that many distinct values, so that many entries share one omega."""
    rng = np.random.default_rng(seed)
    if tie_levels > 0:
        score = rng.integers(0, tie_levels, n).astype(np.float64) / 8.0
    else:
        score = np.exp(3.0 * rng.standard_normal(n))
    depth = rng.integers(0, max_depth + 1, n).astype(np.int32)
    return score, depth


def make_cgee_inputs(B: int, D: int, V: int, seed: int = SEED_BASE + 60, logit_std: float = 3.0, peaked_rows=()):
    """Synthetic inputs of the entropy hook: hidden rows h [B][D] and an unembedding matrix W_u [V][D],
    both bf16 (torch), drawn so that the logits h W_u^T are about N(0, logit_std^2) - an entropy a few nats
    below log V, as for a model some layers into its verify pass.  Rows in ``peaked_rows`` are aligned with
    one vocabulary row each (a concentrated distribution: small entropy, top-1 probability near 1)."""
    gen = _torch_gen(seed, 7)
    w = torch.randn((V, D), generator=gen, dtype=torch.float32) / math.sqrt(D)
    h = torch.randn((B, D), generator=gen, dtype=torch.float32) * logit_std
    for i, b in enumerate(peaked_rows):
        v = (977 * (i + 1)) % V
        h[b] = w[v] * (12.0 / float(w[v].pow(2).sum()))      # that row's logit is 12, the others stay near 0
    return h.to(torch.bfloat16), w.to(torch.bfloat16)


def layer_variant(w: Workload, layer: int) -> Workload:
    """The inputs of another transformer layer of the same decode step: the tables (and so the page
    ids, token counts and sharing) are the step's, the numbers are the layer's own.  Layer 0 is ``w``;
    layer l > 0 holds w's values moved around - keys rotated by l along head_dim, values by 3 l + 1,
    queries by l along the branch axis - so that every layer has a different result while the
    sentinel in the unused slots of partial pages stays where it is.  Works on host or device tensors."""
    if layer == 0:
        return w
    d = w.layout.head_dim
    return dataclasses.replace(
        w, name=f"{w.name}/layer{layer}",
        q=torch.roll(w.q, shifts=layer, dims=0).contiguous(),
        k_pool=torch.roll(w.k_pool, shifts=layer % d, dims=-1).contiguous(),
        v_pool=torch.roll(w.v_pool, shifts=(3 * layer + 1) % d, dims=-1).contiguous())


def make_config(name: str, **kw) -> Workload:
    if name == "tiny":
        return make_tiny(**kw)
    if name == "qwen_layer":
        return make_qwen_layer(**kw)
    if name == "tot":
        return make_tot(**kw)
    if name == "batched_serving":
        return make_batched_serving(**kw)
    if name == "long_context":
        return make_long_context(**kw)
    if name == "diverse_phrasing":
        return make_diverse_phrasing(**kw)
    if name == "long_prefix_serving":
        # batched serving with prefixes of 4096-16384 tokens and the paper's short suffixes (s = 16 plus up to
        # 112 decoded tokens): about 2 GB of unique KV, most of it prefixes
        w = make_batched_serving(prefix_range=(4096, 16384), suffix_range=(16, 128), **kw)
        w.name = "long_prefix_serving"
        return w
    raise ValueError(f"unknown config {name!r}; choose from {CONFIG_NAMES}")


# --------------------------------------------------------------------------------------
# byte counts used by the measurement (plain counting of table entries)
# --------------------------------------------------------------------------------------

def _segment_valid_tokens(t: Tables, s: int) -> int:
    return int(t.seg_num_tokens[s])


def unique_kv_bytes(layout: Layout, t: Tables) -> int:
    """Valid tokens of the distinct segments some branch references, times bytes per token."""
    used = np.unique(t.br_segs)
    tokens = int(sum(_segment_valid_tokens(t, int(s)) for s in used))
    return tokens * layout.bytes_per_token


def duplicated_kv_bytes(layout: Layout, t: Tables) -> int:
    """Bytes a per-branch physical copy of prefix + suffix would hold (the paper's broadcast)."""
    tokens = int(sum(_segment_valid_tokens(t, int(s)) for s in t.br_segs))
    return tokens * layout.bytes_per_token
