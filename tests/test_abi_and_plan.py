"""CPU-side checks: the C ABI exports what the header declares; plan host logic; table builder vs oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import workloads
import paper_2606_09937_b200 as rk


def test_library_exports_every_declared_symbol(repo_root):
    hdr = open(os.path.join(repo_root, "include", "rksc.h")).read()
    declared = set(re.findall(r"RKSC_API\s+[\w\s\*]+?\b(rksc_\w+)\s*\(", hdr))
    assert len(declared) >= 12
    lib = ctypes.CDLL(rk.lib_path())
    for name in declared:
        assert hasattr(lib, name), f"{name} is declared in rksc.h but not exported"
    assert declared == set(rk.EXPORTED_SYMBOLS)


def test_strerror_and_error_codes():
    assert rk.rksc_strerror(0) == "ok"
    for code in range(-7, 0):
        assert rk.rksc_strerror(code) not in ("ok", "unknown status")
    assert rk.rksc_strerror(-99) == "unknown status"


def _plan_for(w, tables=None):
    return rk.rksc_plan_create(w.layout, tables if tables is not None else w.tables)


@pytest.mark.parametrize("maker", [
    lambda: workloads.make_tiny(),
    lambda: workloads.make_tot(root_tokens=300, level_tokens=50),
    lambda: workloads.make_from_segments("r", 28, 4, 128, [37, 5, 16, 1, 0, 1000, 17],
                                         [[0, 1], [0, 2], [3], [0, 4, 5], [], [5, 6], [0, 5, 6]], seed=1),
    lambda: workloads.make_from_segments("wide", 8, 8, 128, [5000], [[0]] * 300, seed=2),
])
def test_plan_covers_every_page_row_pair_once(maker):
    w = maker()
    t = w.tables
    p = _plan_for(w)
    L = w.layout
    G = L.num_q_heads // L.num_kv_heads
    sharers = oracle.segment_sharers(t.br_seg_off, t.br_segs, t.num_segments)
    items = p.items()
    seen = {}
    rows_total = 0
    for seg, kvh, p0, npg, ntok, s0, ns, prow, klass, _ in items.tolist():
        assert npg >= 1 and ns >= 1
        assert ns * G <= (128 if klass == 1 else 64)
        if klass == 1:
            assert ns * G >= 9 and L.head_dim == 128        # the tensor-core kernel takes 9..128 stacked rows
        elif L.head_dim == 128:
            assert ns * G <= 8                              # the warp kernel's small-row path
        seg_pages = int(t.seg_block_off[seg + 1] - t.seg_block_off[seg])
        assert p0 + npg <= seg_pages and s0 + ns <= len(sharers[seg])
        assert ntok == min(int(t.seg_num_tokens[seg]), (p0 + npg) * 16) - p0 * 16
        for page in range(p0, p0 + npg):
            for s in range(s0, s0 + ns):
                key = (seg, kvh, page, s)
                assert key not in seen
                seen[key] = True
        rows_total += ns * G
    expect = sum(int(t.seg_block_off[s + 1] - t.seg_block_off[s]) * len(sharers[s]) for s in range(t.num_segments))
    assert len(seen) == expect * L.num_kv_heads
    assert p.num_partial_rows == rows_total
    # partial rows are laid out item after item
    order = np.argsort(items[:, 7], kind="stable")
    ends = items[order, 7] + items[order, 6] * G
    assert np.array_equal(ends[:-1], items[order, 7][1:]) if len(items) > 1 else True
    # masses and token counts agree with the oracle's integer helpers
    assert np.array_equal(p.mass_off, oracle.mass_offsets(t.seg_block_off, t.br_seg_off, t.br_segs))
    assert p.mass_elems == int(p.mass_off[-1]) * L.num_q_heads
    assert p.unique_kv_tokens * L.bytes_per_token == workloads.unique_kv_bytes(L, t)
    assert p.duplicated_kv_tokens * L.bytes_per_token == workloads.duplicated_kv_bytes(L, t)
    assert p.workspace_bytes >= p.num_partial_rows * (L.head_dim + 1) * 4


def test_plan_rejects_bad_tables_and_layouts():
    w = workloads.make_tiny()
    t = w.tables

    def create(layout=None, **over):
        d = {k: getattr(t, k).copy() for k in ("seg_block_off", "seg_blocks", "seg_num_tokens", "br_seg_off", "br_segs")}
        d.update(over)
        return rk.rksc_plan_create(layout or w.layout, d)

    bad = t.seg_blocks.copy(); bad[3] = w.layout.num_pool_blocks
    with pytest.raises(rk.RkscError) as e:
        create(seg_blocks=bad)
    assert e.value.status == -3
    bad = t.seg_blocks.copy(); bad[0] = -1
    with pytest.raises(rk.RkscError):
        create(seg_blocks=bad)
    nt = t.seg_num_tokens.copy(); nt[0] = 257          # more tokens than 16 pages hold
    with pytest.raises(rk.RkscError) as e:
        create(seg_num_tokens=nt)
    assert e.value.status == -3
    nt = t.seg_num_tokens.copy(); nt[0] = 240          # last listed page would be empty
    with pytest.raises(rk.RkscError):
        create(seg_num_tokens=nt)
    bs = t.br_segs.copy(); bs[0] = t.num_segments
    with pytest.raises(rk.RkscError):
        create(br_segs=bs)
    import dataclasses
    with pytest.raises(rk.RkscError) as e:
        create(layout=dataclasses.replace(w.layout, head_dim=96))
    assert e.value.status == -2
    with pytest.raises(rk.RkscError) as e:
        create(layout=dataclasses.replace(w.layout, num_q_heads=7))
    assert e.value.status == -1
    with pytest.raises(rk.RkscError) as e:
        create(layout=dataclasses.replace(w.layout, block_size=32))
    assert e.value.status == -2


def test_tables_from_gate_matches_oracle_on_random_maps():
    rng = np.random.default_rng(3)
    w = workloads.make_batched_serving(problems=6, branches_per=5, prefix_range=(1, 90), suffix_range=(0, 40),
                                       L=2, D=64, head_dim=64, num_q_heads=4, num_kv_heads=2, perturbed_frac=0.4)
    f = w.flat
    B = w.num_branches
    for trial in range(20):
        m = np.array([b // 5 if rng.random() < 0.6 else -1 for b in range(B)], dtype=np.int32)
        if trial == 0:
            m[:] = -1
        if trial == 1:
            m = np.array([b // 5 for b in range(B)], dtype=np.int32)
        args = (m, f.num_prefixes, f.shared_off, f.shared_pages, f.shared_ntok, f.priv_off, f.priv_pages,
                f.priv_ntok, f.sfx_off, f.sfx_pages, f.sfx_ntok)
        got = rk.rksc_tables_from_gate(*args).as_dict()
        ref = oracle.tables_from_gate(*args)
        for k in ref:
            assert np.array_equal(got[k], ref[k]), (trial, k)
    with pytest.raises(rk.RkscError):
        m = np.zeros(B, dtype=np.int32); m[0] = f.num_prefixes      # map entry out of range
        rk.rksc_tables_from_gate(m, f.num_prefixes, f.shared_off, f.shared_pages, f.shared_ntok, f.priv_off,
                                 f.priv_pages, f.priv_ntok, f.sfx_off, f.sfx_pages, f.sfx_ntok)


def test_compute_calls_fail_loudly_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    w = workloads.make_tiny()
    p = _plan_for(w)
    assert not p.on_device
    buf = (ctypes.c_char * 4096)()
    st = rk.lib().rksc_branch_decode_attention(p._h, buf, buf, buf, buf, None, None, 0, None, None)
    assert st in (-4, -5)          # no workspace / no device: never a silent success
    hb = np.zeros((1, 1, 4), np.float32)
    st = rk.lib().rksc_asks_gate(hb.ctypes.data, hb.ctypes.data, hb.ctypes.data, 1, 1, 1, 4, 0.5, 0.9,
                                 hb.ctypes.data, None, None)
    assert st == -5
