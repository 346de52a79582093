"""Pins for the suffix-prefill oracle (Section 2.2; Appendix "Stepwise Batched Decode", step 1)."""
import numpy as np
import pytest

import oracle
import workloads


def _args(w, t=None):
    t = w.tables if t is None else t
    get = (lambda k: t[k]) if isinstance(t, dict) else (lambda k: getattr(t, k))
    L = w.layout
    return (L.num_q_heads, L.num_kv_heads, L.head_dim, L.sm_scale, get("seg_block_off"), get("seg_blocks"),
            get("seg_num_tokens"), get("br_seg_off"), get("br_segs"))


def _small(seed=3, hq=4, hkv=2, d=64):
    # a shared prefix of 37 tokens, suffixes of 21, 40 and 16 tokens (the last: exactly s tokens for s = 16)
    return workloads.make_from_segments("sp", hq, hkv, d, [37, 21, 40, 16], [[0, 1], [0, 2], [0, 3]], seed=seed)


def _queries(w, s, seed=5):
    rng = np.random.default_rng(seed)
    L = w.layout
    return rng.standard_normal((w.tables.num_branches, s, L.num_q_heads, L.head_dim))


def test_one_token_is_decode_attention():
    w = _small()
    q = _queries(w, 1)
    pools = (oracle.to_f32_numpy(w.k_pool), oracle.to_f32_numpy(w.v_pool))
    out, m = oracle.suffix_prefill_attention(*_args(w), q, *pools)
    ref, rm = oracle.branch_decode_attention(*_args(w), q[:, 0], *pools)
    assert np.array_equal(out[:, 0], ref)
    for b in range(3):
        assert np.array_equal(m[b][0], rm[b])


def test_last_token_sees_everything_and_rows_sum_to_one():
    w = _small()
    s = 5
    q = _queries(w, s)
    pools = (oracle.to_f32_numpy(w.k_pool), oracle.to_f32_numpy(w.v_pool))
    out, m = oracle.suffix_prefill_attention(*_args(w), q, *pools)
    ref, rm = oracle.branch_decode_attention(*_args(w), q[:, s - 1], *pools)
    assert np.allclose(out[:, s - 1], ref, rtol=0, atol=1e-14)
    for b in range(3):
        assert np.allclose(m[b].sum(axis=2), 1.0, atol=1e-12)
        assert np.allclose(m[b][s - 1], rm[b], atol=1e-14)


def test_causal_later_tokens_do_not_matter():
    w = _small()
    s = 6
    q = _queries(w, s)
    k = oracle.to_f32_numpy(w.k_pool).copy()
    v = oracle.to_f32_numpy(w.v_pool).copy()
    out, _ = oracle.suffix_prefill_attention(*_args(w), q, k, v)
    # overwrite the keys and values of the last 3 tokens of branch 1's suffix (40 tokens: pages 2 of its segment)
    t = w.tables
    seg = int(t.br_segs[t.br_seg_off[1] + 1])
    page = int(t.seg_blocks[t.seg_block_off[seg] + 2])      # tokens 32..39
    k[page, :, 5:8, :] = 9.0
    v[page, :, 5:8, :] = -9.0
    out2, _ = oracle.suffix_prefill_attention(*_args(w), q, k, v)
    assert np.array_equal(out2[1, :3], out[1, :3])           # tokens 0..2 stand before the changed positions
    assert not np.allclose(out2[1, 3:], out[1, 3:])
    assert np.array_equal(out2[0], out[0]) and np.array_equal(out2[2], out[2])


def test_scalar_loop_twin():
    w = _small(hq=2, hkv=1, d=64)
    s = 3
    q = _queries(w, s)
    k, v = oracle.to_f32_numpy(w.k_pool).astype(np.float64), oracle.to_f32_numpy(w.v_pool).astype(np.float64)
    out, _ = oracle.suffix_prefill_attention(*_args(w), q, k, v)
    t = w.tables
    b, i, h = 1, 1, 1
    toks = []
    for sgi in t.br_segs[t.br_seg_off[b]:t.br_seg_off[b + 1]]:
        for p, page in enumerate(t.seg_blocks[t.seg_block_off[sgi]:t.seg_block_off[sgi + 1]]):
            for j in range(min(16, int(t.seg_num_tokens[sgi]) - 16 * p)):
                toks.append((int(page), j))
    T = len(toks)
    toks = toks[:T - s + i + 1]
    scale = 1.0 / np.sqrt(64.0)
    logits = [scale * sum(float(q[b, i, h, c]) * k[pg, 0, j, c] for c in range(64)) for pg, j in toks]
    mx = max(logits)
    e = [np.exp(x - mx) for x in logits]
    Z = sum(e)
    ref = [sum(e[n] * v[pg, 0, j, c] for n, (pg, j) in enumerate(toks)) / Z for c in range(64)]
    assert np.allclose(out[b, i, h], ref, atol=1e-12)


def test_tables_hand_case():
    # one branch: prefix segment 0 (20 tokens, pages 7, 8) + own segment 1 (35 tokens, pages 3, 4, 5); s = 4:
    # the 4 tokens are positions 31..34 of segment 1 -> one page (16 tokens) lies wholly before them
    t = oracle.suffix_prefill_tables([0, 2, 5], [7, 8, 3, 4, 5], [20, 35], [0, 2], [0, 1], 4)
    assert t["seg_block_off"].tolist() == [0, 2, 5, 6, 7, 9, 11, 13]
    assert t["seg_blocks"].tolist() == [7, 8, 3, 4, 5, 3, 4, 4, 5, 4, 5, 4, 5]
    assert t["seg_num_tokens"].tolist() == [20, 35, 16, 16, 17, 18, 19]
    assert t["br_seg_off"].tolist() == [0, 3, 6, 9, 12]
    assert t["br_segs"].tolist() == [0, 2, 3, 0, 2, 4, 0, 2, 5, 0, 2, 6]
    with pytest.raises(ValueError):
        oracle.suffix_prefill_tables([0, 2, 5], [7, 8, 3, 4, 5], [20, 3], [0, 2], [0, 1], 4)


@pytest.mark.parametrize("s", [1, 4, 16])
def test_decode_attention_over_virtual_tables_is_the_suffix_prefill(s):
    w = _small()
    q = _queries(w, s)
    pools = (oracle.to_f32_numpy(w.k_pool), oracle.to_f32_numpy(w.v_pool))
    out, m = oracle.suffix_prefill_attention(*_args(w), q, *pools)
    t = w.tables
    vt = oracle.suffix_prefill_tables(t.seg_block_off, t.seg_blocks, t.seg_num_tokens, t.br_seg_off, t.br_segs, s)
    B = t.num_branches
    vout, vm = oracle.branch_decode_attention(*_args(w, vt), q.reshape(B * s, *q.shape[2:]), *pools)
    assert np.allclose(vout.reshape(out.shape), out, rtol=0, atol=1e-14)
    for b in range(B):
        for i in range(s):
            n = vm[b * s + i].shape[1]               # the leading blocks of the branch
            assert n <= m[b][i].shape[1]
            assert np.allclose(vm[b * s + i], m[b][i][:, :n], atol=1e-14)
            assert np.all(m[b][i][:, n:] == 0)
