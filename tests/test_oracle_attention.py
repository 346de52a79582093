"""Pins for the attention oracle: closed forms, brute force, invariants."""
import math
from decimal import Decimal, getcontext

import numpy as np
import pytest
import scipy.special
import torch

import oracle
import workloads
from workloads import Tables
from helpers import oracle_attention

getcontext().prec = 40


def _segs(w, b):
    t = w.tables
    return t.br_segs[t.br_seg_off[b]:t.br_seg_off[b + 1]]


def _logical_kv(w, b):
    """Independent gather with torch indexing: valid tokens of branch b as [T][Hkv][d] fp64."""
    t = w.tables
    ks, vs = [], []
    for s in _segs(w, b):
        pages = torch.from_numpy(t.seg_blocks[t.seg_block_off[s]:t.seg_block_off[s + 1]].astype(np.int64))
        n = int(t.seg_num_tokens[s])
        k = w.k_pool[pages].permute(0, 2, 1, 3).reshape(-1, w.layout.num_kv_heads, w.layout.head_dim)[:n]
        v = w.v_pool[pages].permute(0, 2, 1, 3).reshape(-1, w.layout.num_kv_heads, w.layout.head_dim)[:n]
        ks.append(k.double().numpy()); vs.append(v.double().numpy())
    return np.concatenate(ks), np.concatenate(vs)


def test_against_scipy_softmax_with_partial_pages_and_gqa():
    # ragged lengths so that sentinel slots exist; 6 q heads on 2 kv heads (G = 3)
    w = workloads.make_from_segments("r", 6, 2, 64, [37, 5, 16, 1], [[0, 1], [0, 2], [3]], seed=1)
    out, masses = oracle_attention(w)
    for b in range(3):
        K, V = _logical_kv(w, b)
        for h in range(6):
            g = h // 3
            s = (K[:, g, :] @ w.q[b, h].double().numpy()) / math.sqrt(64)
            p = scipy.special.softmax(s)
            assert np.allclose(out[b, h], p @ V[:, g, :], rtol=0, atol=1e-13)
            # masses: reduce p over 16-token pages of each segment separately
            j = 0; pos = 0
            for sgm in _segs(w, b):
                n = int(w.tables.seg_num_tokens[sgm])
                for lo in range(0, n, 16):
                    hi = min(n, lo + 16)
                    assert abs(masses[b][h, j] - p[pos + lo:pos + hi].sum()) < 1e-14
                    j += 1
                pos += n
            assert j == masses[b].shape[1]
    assert np.abs(out).max() < 10  # no sentinel leaked


def test_brute_force_twin_decimal():
    w = workloads.make_from_segments("b", 2, 1, 64, [19, 3], [[0, 1], [0]], seed=2)
    out, masses = oracle_attention(w)
    for b in range(2):
        K, V = _logical_kv(w, b)
        T = K.shape[0]
        for h in range(2):
            qv = w.q[b, h].double().numpy()
            # no max subtraction, token-major loops, exact exp in decimal
            e = []
            for j in range(T):
                s = sum(Decimal(float(qv[k])) * Decimal(float(K[j, 0, k])) for k in range(64))
                e.append((s / Decimal(64).sqrt()).exp())
            z = sum(e)
            for k in range(0, 64, 7):
                ref = sum(e[j] / z * Decimal(float(V[j, 0, k])) for j in range(T))
                assert abs(out[b, h, k] - float(ref)) < 1e-13
            assert abs(masses[b][h, 0] - float(sum(e[:16]) / z)) < 1e-13


def _custom(K, V, q, seg_ntok, br_segs, Hq, Hkv, d, sm_scale=0.0):
    """Workload from explicit logical K/V ([T_total][Hkv][d] per segment concatenated)."""
    w = workloads.make_from_segments("c", Hq, Hkv, d, seg_ntok, br_segs, seed=9, sm_scale=sm_scale)
    t = w.tables
    pos = 0
    for s, n in enumerate(seg_ntok):
        for i, page in enumerate(t.seg_blocks[t.seg_block_off[s]:t.seg_block_off[s + 1]]):
            lo, hi = 16 * i, min(n, 16 * i + 16)
            w.k_pool[int(page), :, : hi - lo, :] = torch.as_tensor(K[pos + lo:pos + hi]).permute(1, 0, 2).to(torch.bfloat16)
            w.v_pool[int(page), :, : hi - lo, :] = torch.as_tensor(V[pos + lo:pos + hi]).permute(1, 0, 2).to(torch.bfloat16)
        pos += n
    w.q = torch.as_tensor(q).to(torch.bfloat16)
    return w


def _bf(x):
    return torch.as_tensor(x, dtype=torch.float32).to(torch.bfloat16).double().numpy()


def test_identical_keys_give_mean_of_v_and_uniform_mass():
    rng = np.random.default_rng(3)
    T, d = 41, 64
    k0 = rng.standard_normal((1, 2, d))
    K = np.repeat(k0, T, axis=0)
    V = _bf(rng.standard_normal((T, 2, d)))
    q = rng.standard_normal((1, 4, d))
    w = _custom(K, V, q, [T], [[0]], 4, 2, d)
    out, masses = oracle_attention(w)
    for h in range(4):
        assert np.allclose(out[0, h], V[:, h // 2, :].mean(axis=0), atol=1e-13)   # also pins h -> h // G
        assert np.allclose(masses[0][h], np.array([16, 16, 9]) / T, atol=1e-14)


def test_single_token_zero_query_two_tokens_one_hot():
    rng = np.random.default_rng(4)
    d = 64
    K = _bf(rng.standard_normal((2, 1, d)))
    V = _bf(rng.standard_normal((2, 1, d)))
    q = _bf(rng.standard_normal((1, 1, d)))
    # T = 1: out = V_0
    out, m = oracle_attention(_custom(K[:1], V[:1], q, [1], [[0]], 1, 1, d))
    assert np.array_equal(out[0, 0], V[0, 0]) and m[0][0, 0] == 1.0
    # q = 0: uniform
    out, _ = oracle_attention(_custom(K, V, np.zeros((1, 1, d)), [2], [[0]], 1, 1, d))
    assert np.allclose(out[0, 0], V[:, 0].mean(axis=0), atol=1e-15)
    # two tokens: p_1 = sigmoid(s_1 - s_2) with s = q.k / sqrt(d); and with a custom scale
    for scale, eff in ((0.0, 1 / math.sqrt(d)), (0.37, float(np.float32(0.37)))):
        out, m = oracle_attention(_custom(K, V, q, [2], [[0]], 1, 1, d, sm_scale=scale))
        s = (K[:, 0] @ q[0, 0]) * eff
        p1 = 1 / (1 + math.exp(-(s[0] - s[1])))
        assert np.allclose(out[0, 0], p1 * V[0, 0] + (1 - p1) * V[1, 0], atol=1e-14)
    # one key aligned with q and scaled x50: one-hot on that token
    T = 20
    K = _bf(rng.standard_normal((T, 1, d)))
    V = _bf(rng.standard_normal((T, 1, d)))
    K[7, 0] = _bf(50 * q[0, 0] / np.linalg.norm(q[0, 0]) * math.sqrt(d))
    out, m = oracle_attention(_custom(K, V, q, [T], [[0]], 1, 1, d))
    assert np.allclose(out[0, 0], V[7, 0], atol=1e-9) and abs(m[0][0, 0] - 1) < 1e-9


def test_key_shift_invariance():
    rng = np.random.default_rng(5)
    T, d = 30, 64
    K = rng.integers(-8, 8, (T, 1, d)).astype(np.float64) / 4      # exactly representable
    V = _bf(rng.standard_normal((T, 1, d)))
    q = rng.integers(-8, 8, (1, 2, d)).astype(np.float64) / 4
    c = rng.integers(-8, 8, (1, 1, d)).astype(np.float64) / 4
    o1, m1 = oracle_attention(_custom(K, V, q, [T], [[0]], 2, 1, d))
    o2, m2 = oracle_attention(_custom(K + c, V, q, [T], [[0]], 2, 1, d))
    assert np.allclose(o1, o2, atol=1e-12) and np.allclose(m1[0], m2[0], atol=1e-12)


def _duplicate_physically(w):
    """Same logical data, but every branch gets its own physical copy of every segment."""
    t = w.tables
    new_blocks, new_off, new_ntok, br_segs = [], [0], [], []
    pages_k, pages_v = [], []
    for b in range(t.num_branches):
        mine = []
        for s in t.br_segs[t.br_seg_off[b]:t.br_seg_off[b + 1]]:
            src = t.seg_blocks[t.seg_block_off[s]:t.seg_block_off[s + 1]]
            base = len(new_blocks)
            new_blocks += list(range(base, base + len(src)))
            new_off.append(len(new_blocks)); new_ntok.append(int(t.seg_num_tokens[s]))
            idx = torch.from_numpy(src.astype(np.int64))
            pages_k.append(w.k_pool[idx]); pages_v.append(w.v_pool[idx])
            mine.append(len(new_ntok) - 1)
        br_segs.append(mine)
    off = np.zeros(len(br_segs) + 1, np.int32); off[1:] = np.cumsum([len(x) for x in br_segs])
    nt = Tables(np.array(new_off, np.int32), np.array(new_blocks, np.int32), np.array(new_ntok, np.int32),
                off, np.array([s for x in br_segs for s in x], np.int32))
    import dataclasses
    return dataclasses.replace(w, k_pool=torch.cat(pages_k), v_pool=torch.cat(pages_v), tables=nt)


def test_shared_tables_equal_duplicated_tables():
    w = workloads.make_tot(head_dim=64, num_q_heads=4, num_kv_heads=2, root_tokens=50,
                           level_tokens=21, branching=2, depth=2)
    o1, m1 = oracle_attention(w)
    o2, m2 = oracle_attention(_duplicate_physically(w))
    assert np.array_equal(o1, o2)
    assert all(np.array_equal(a, b) for a, b in zip(m1, m2))


def test_page_permutation_and_segment_split():
    w = workloads.make_from_segments("p", 4, 2, 64, [64, 20], [[0, 1], [0]], seed=6)
    o1, m1 = oracle_attention(w)
    t = w.tables
    perm = np.array([2, 0, 3, 1])
    blocks = t.seg_blocks.copy(); blocks[:4] = t.seg_blocks[:4][perm]
    import dataclasses
    w2 = dataclasses.replace(w, tables=dataclasses.replace(t, seg_blocks=blocks))
    o2, m2 = oracle_attention(w2)
    assert np.allclose(o1, o2, atol=1e-14)
    assert np.allclose(m2[0][:, :4], m1[0][:, perm], atol=1e-15)
    assert np.allclose(m2[0][:, 4:], m1[0][:, 4:], atol=1e-15)
    # split segment 0 (4 full pages) into 1 + 3 pages: nothing changes
    t3 = Tables(np.array([0, 1, 4, 6], np.int32), t.seg_blocks, np.array([16, 48, 20], np.int32),
                np.array([0, 3, 5], np.int32), np.array([0, 1, 2, 0, 1], np.int32))
    o3, m3 = oracle_attention(dataclasses.replace(w, tables=t3))
    assert np.allclose(o1, o3, atol=1e-14) and np.allclose(m1[0], m3[0], atol=1e-15)


def test_masses_sum_to_one_and_eviction_renormalises():
    w = workloads.make_long_context(prefix=400, suffix=40, branches=3, num_q_heads=4,
                                    num_kv_heads=2, head_dim=64)
    o, m = oracle_attention(w)
    for b in range(3):
        assert np.allclose(m[b].sum(axis=1), 1.0, atol=1e-13)
    scores = sum(mb[:, :25].sum(axis=0) for mb in m)
    ev = workloads.lowest_mass_pages(scores, 0.2)
    assert len(ev) == 5
    h = workloads.punch_holes(w, 0, ev)
    o2, m2 = oracle_attention(h)
    keep = np.setdiff1d(np.arange(m[0].shape[1]), ev)
    for b in range(3):
        gone = m[b][:, ev].sum(axis=1, keepdims=True)
        assert np.allclose(m2[b], m[b][:, keep] / (1 - gone), atol=1e-13)


def test_empty_branch_and_empty_segment():
    w = workloads.make_from_segments("e", 2, 1, 64, [0, 18], [[0], [0, 1], []], seed=7)
    o, m = oracle_attention(w)
    assert np.all(o[0] == 0) and m[0].shape == (2, 0)
    assert np.all(o[2] == 0) and m[2].shape == (2, 0)
    assert m[1].shape == (2, 2) and np.allclose(m[1].sum(axis=1), 1)


def test_output_scale_matches_error_budget():
    # N(0,1) data: output elements ~ N(0, e/T)
    w = workloads.make_tiny()
    o, _ = oracle_attention(w)
    assert 0.08 < o.std() < 0.12
