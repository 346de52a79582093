"""ctypes binding of librksc.so: argument marshalling only.

Every function mirrors the C entry point of the same name (see include/rksc.h).
Tensors are torch CUDA tensors whose data pointers are handed to the library;
work is enqueued on torch's current stream unless a stream is given.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

import numpy as np

_PKG_DIR = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_PKG_DIR, "librksc.so")
_lib = None

EXPORTED_SYMBOLS = (
    "rksc_strerror",
    "rksc_last_cuda_error",
    "rksc_asks_gate",
    "rksc_tables_from_gate",
    "rksc_tables_free",
    "rksc_plan_create",
    "rksc_plan_create_from_gate",
    "rksc_plan_query",
    "rksc_plan_get_item",
    "rksc_plan_destroy",
    "rksc_branch_decode_attention",
    "rksc_branch_decode_attention_phases",
    "rksc_branch_decode_attention_static",
    "rksc_decode_step_host",
    "rksc_rsbcm_page_scores",
    "rksc_rsbcm_workspace_bytes",
    "rksc_rsbcm_evict",
    "rksc_tables_drop_evicted",
    "rksc_tables_for_suffix_prefill",
    "rksc_tables_append_token",
    "rksc_kv_append",
    "rksc_cgee_workspace_bytes",
    "rksc_cgee_logit_entropy",
    "rksc_cgee_entropy_exit",
    "rksc_cgee_verify_skip",
    "rksc_debug_wait_timeout",
    "rksc_pipeline_create",
    "rksc_pipeline_submit",
    "rksc_pipeline_wait",
    "rksc_pipeline_destroy",
)
STATIC_WORKSPACE_BYTES = 16 << 20


class RkscError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = int(status)
        detail = ""
        if status == -5:
            detail = " [" + lib().rksc_last_cuda_error().decode() + "]"
        super().__init__(f"{where}: {rksc_strerror(status)} (status {status}){detail}")


class _CLayout(C.Structure):
    _fields_ = [("num_q_heads", C.c_int32), ("num_kv_heads", C.c_int32), ("head_dim", C.c_int32),
                ("block_size", C.c_int32), ("sm_scale", C.c_float), ("num_pool_blocks", C.c_int32)]


class _CTables(C.Structure):
    _fields_ = [("num_branches", C.c_int32), ("num_segments", C.c_int32),
                ("seg_block_off", C.POINTER(C.c_int32)), ("seg_blocks", C.POINTER(C.c_int32)),
                ("seg_num_tokens", C.POINTER(C.c_int32)), ("br_seg_off", C.POINTER(C.c_int32)),
                ("br_segs", C.POINTER(C.c_int32))]


class _CPlanInfo(C.Structure):
    _fields_ = [("workspace_bytes", C.c_size_t), ("mass_elems", C.c_int64),
                ("mass_off", C.POINTER(C.c_int64)), ("num_work_items", C.c_int32),
                ("num_partial_rows", C.c_int32), ("unique_kv_tokens", C.c_int64),
                ("duplicated_kv_tokens", C.c_int64), ("on_device", C.c_int32), ("num_pages_listed", C.c_int64),
                ("num_kernel_launches", C.c_int32)]


def lib_path() -> str:
    return _LIB_PATH


def lib() -> C.CDLL:
    """The loaded library.  Raises if it has not been built (there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_2606_09937_b200.build` "
            "(needs nvcc).  This package has no CPU or eager fallback.")
    L = C.CDLL(_LIB_PATH)
    i32p = C.POINTER(C.c_int32)
    L.rksc_strerror.restype = C.c_char_p
    L.rksc_strerror.argtypes = [C.c_int32]
    L.rksc_last_cuda_error.restype = C.c_char_p
    L.rksc_last_cuda_error.argtypes = []
    L.rksc_asks_gate.restype = C.c_int32
    L.rksc_asks_gate.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32,
                                 C.c_int32, C.c_float, C.c_float, C.c_void_p, C.c_void_p, C.c_void_p]
    L.rksc_tables_from_gate.restype = C.c_int32
    L.rksc_tables_from_gate.argtypes = [C.c_int32, C.c_int32, i32p] + [i32p] * 9 + [C.POINTER(_CTables)]
    L.rksc_tables_free.restype = None
    L.rksc_tables_free.argtypes = [C.POINTER(_CTables)]
    L.rksc_plan_create.restype = C.c_int32
    L.rksc_plan_create.argtypes = [C.POINTER(_CLayout), C.POINTER(_CTables), C.POINTER(C.c_void_p)]
    L.rksc_plan_create_from_gate.restype = C.c_int32
    L.rksc_plan_create_from_gate.argtypes = [C.POINTER(_CLayout), C.c_int32, C.c_int32] + [i32p] * 10 + [C.POINTER(C.c_void_p)]
    L.rksc_plan_query.restype = C.c_int32
    L.rksc_plan_query.argtypes = [C.c_void_p, C.POINTER(_CPlanInfo)]
    L.rksc_plan_get_item.restype = C.c_int32
    L.rksc_plan_get_item.argtypes = [C.c_void_p, C.c_int32, i32p]
    L.rksc_plan_destroy.restype = None
    L.rksc_plan_destroy.argtypes = [C.c_void_p]
    L.rksc_branch_decode_attention.restype = C.c_int32
    L.rksc_branch_decode_attention.argtypes = [C.c_void_p] * 7 + [C.c_size_t, C.c_void_p, C.c_void_p]
    L.rksc_branch_decode_attention_phases.restype = C.c_int32
    L.rksc_branch_decode_attention_phases.argtypes = [C.c_void_p] * 7 + [C.c_size_t, C.c_void_p, C.c_void_p, C.c_int32]
    L.rksc_decode_step_host.restype = C.c_int32
    L.rksc_decode_step_host.argtypes = ([C.POINTER(_CLayout), C.c_void_p, C.c_void_p, C.c_void_p] + [C.c_int32] * 4 +
                                        [C.c_float, C.c_float] + [i32p] * 9 + [C.c_void_p] * 7 +
                                        [C.c_int64, C.c_void_p, C.c_void_p])
    L.rksc_branch_decode_attention_static.restype = C.c_int32
    L.rksc_branch_decode_attention_static.argtypes = [C.c_void_p] * 8
    L.rksc_rsbcm_page_scores.restype = C.c_int32
    L.rksc_rsbcm_page_scores.argtypes = [C.c_void_p] * 4
    L.rksc_rsbcm_workspace_bytes.restype = C.c_size_t
    L.rksc_rsbcm_workspace_bytes.argtypes = [C.c_int64]
    L.rksc_rsbcm_evict.restype = C.c_int32
    L.rksc_rsbcm_evict.argtypes = [C.c_void_p, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p,
                                   C.c_size_t, C.c_void_p]
    L.rksc_tables_append_token.restype = C.c_int32
    L.rksc_tables_append_token.argtypes = [C.POINTER(_CTables), i32p, C.POINTER(_CTables), i32p, i32p]
    L.rksc_kv_append.restype = C.c_int32
    L.rksc_kv_append.argtypes = [C.POINTER(_CLayout)] + [C.c_void_p] * 4 + [C.c_int32, C.c_void_p, C.c_void_p, C.c_void_p]
    L.rksc_cgee_workspace_bytes.restype = C.c_size_t
    L.rksc_cgee_workspace_bytes.argtypes = []
    L.rksc_cgee_logit_entropy.restype = C.c_int32
    L.rksc_cgee_logit_entropy.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int64, C.c_void_p, C.c_void_p,
                                          C.c_void_p, C.c_size_t, C.c_void_p, C.c_void_p]
    L.rksc_cgee_entropy_exit.restype = C.c_int32
    L.rksc_cgee_entropy_exit.argtypes = [C.c_void_p, C.c_void_p, C.c_int32, C.c_int32, C.c_int32, C.c_float, C.c_float,
                                         C.c_void_p, C.c_void_p]
    L.rksc_cgee_verify_skip.restype = C.c_int32
    L.rksc_cgee_verify_skip.argtypes = [C.c_void_p, C.c_int32, C.c_int32, C.c_float, C.c_float, C.c_void_p, C.c_void_p,
                                        C.c_void_p]
    L.rksc_tables_for_suffix_prefill.restype = C.c_int32
    L.rksc_tables_for_suffix_prefill.argtypes = [C.POINTER(_CTables), C.c_int32, C.POINTER(_CTables)]
    L.rksc_tables_drop_evicted.restype = C.c_int32
    L.rksc_tables_drop_evicted.argtypes = [C.POINTER(_CTables), C.c_void_p, C.POINTER(_CTables)]
    L.rksc_debug_wait_timeout.restype = C.c_int32
    L.rksc_debug_wait_timeout.argtypes = [C.c_int64, C.c_void_p, C.c_void_p]
    L.rksc_pipeline_create.restype = C.c_int32
    L.rksc_pipeline_create.argtypes = ([C.POINTER(_CLayout)] + [C.c_int32] * 4 + [C.c_float, C.c_float] + [i32p] * 9 +
                                       [C.c_int32, C.c_int64, C.c_int32, C.POINTER(C.c_void_p)])
    L.rksc_pipeline_submit.restype = C.c_int32
    L.rksc_pipeline_submit.argtypes = [C.c_void_p] * 10 + [C.POINTER(C.c_int64)]
    L.rksc_pipeline_wait.restype = C.c_int32
    L.rksc_pipeline_wait.argtypes = [C.c_void_p, C.c_int64, C.c_void_p, C.c_void_p, C.c_void_p, C.POINTER(_CPlanInfo),
                                     C.POINTER(C.c_float)]
    L.rksc_pipeline_destroy.restype = None
    L.rksc_pipeline_destroy.argtypes = [C.c_void_p]
    _lib = L
    return L


def rksc_strerror(status: int) -> str:
    return lib().rksc_strerror(int(status)).decode()


def _check(status: int, where: str):
    if status != 0:
        raise RkscError(status, where)


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _p(a: np.ndarray):
    return a.ctypes.data_as(C.POINTER(C.c_int32))


def _stream_ptr(stream, device=None) -> int:
    """Raw cudaStream_t of ``stream`` (a torch stream), or of torch's current stream on ``device``."""
    import torch
    if stream is not None:
        return int(stream.cuda_stream)
    idx = device.index if (device is not None and device.index is not None) else torch.cuda.current_device()
    try:
        return int(torch._C._cuda_getCurrentRawStream(idx))   # cheap; the public call re-probes the driver
    except AttributeError:
        return int(torch.cuda.current_stream(idx).cuda_stream)


class Layout:
    """Mirror of rksc_layout."""

    def __init__(self, num_q_heads, num_kv_heads, head_dim, num_pool_blocks, sm_scale=0.0, block_size=16):
        self.c = _CLayout(int(num_q_heads), int(num_kv_heads), int(head_dim), int(block_size),
                          float(sm_scale), int(num_pool_blocks))

    @classmethod
    def of(cls, layout) -> "Layout":
        """From any object with the same attribute names (e.g. a workload's layout)."""
        return cls(layout.num_q_heads, layout.num_kv_heads, layout.head_dim, layout.num_pool_blocks,
                   getattr(layout, "sm_scale", 0.0), getattr(layout, "block_size", 16))


class Tables:
    """Mirror of rksc_tables over host arrays (numpy int32, kept alive here)."""

    def __init__(self, seg_block_off, seg_blocks, seg_num_tokens, br_seg_off, br_segs, _owned=None):
        self.seg_block_off = _i32(seg_block_off)
        self.seg_blocks = _i32(seg_blocks)
        self.seg_num_tokens = _i32(seg_num_tokens)
        self.br_seg_off = _i32(br_seg_off)
        self.br_segs = _i32(br_segs)
        self.c = _CTables(len(self.br_seg_off) - 1, len(self.seg_num_tokens),
                          _p(self.seg_block_off), _p(self.seg_blocks), _p(self.seg_num_tokens),
                          _p(self.br_seg_off), _p(self.br_segs))

    @classmethod
    def of(cls, t) -> "Tables":
        if isinstance(t, cls):
            return t
        if isinstance(t, dict):
            return cls(t["seg_block_off"], t["seg_blocks"], t["seg_num_tokens"], t["br_seg_off"], t["br_segs"])
        return cls(t.seg_block_off, t.seg_blocks, t.seg_num_tokens, t.br_seg_off, t.br_segs)

    def as_dict(self):
        return {k: getattr(self, k) for k in
                ("seg_block_off", "seg_blocks", "seg_num_tokens", "br_seg_off", "br_segs")}


class _OwnedView(np.ndarray):
    """A view of memory another object owns; ``_owner`` keeps that object alive as long as the view
    (or anything sliced from it) is."""


class LibTables(Tables):
    """An rksc_tables the library allocated (rksc_tables_from_gate and the other table calls): kept as
    it is and freed with this object, so that handing it to the next call costs no copy.  The array
    attributes are views of the library's memory, made on access; each keeps this object alive."""

    _FIELDS = {"seg_block_off": ("num_segments", 1), "seg_num_tokens": ("num_segments", 0),
               "br_seg_off": ("num_branches", 1)}

    def __init__(self, c: "_CTables"):
        self.c = c

    def _view(self, name):
        c = self.c
        if name in self._FIELDS:
            count, extra = self._FIELDS[name]
            n = int(getattr(c, count)) + extra
        elif name == "seg_blocks":
            n = int(c.seg_block_off[c.num_segments])
        else:   # br_segs
            n = int(c.br_seg_off[c.num_branches])
        if n <= 0:
            return np.zeros(0, dtype=np.int32)
        v = np.ctypeslib.as_array(getattr(c, name), shape=(n,)).view(_OwnedView)
        v._owner = self
        return v

    seg_block_off = property(lambda self: self._view("seg_block_off"))
    seg_blocks = property(lambda self: self._view("seg_blocks"))
    seg_num_tokens = property(lambda self: self._view("seg_num_tokens"))
    br_seg_off = property(lambda self: self._view("br_seg_off"))
    br_segs = property(lambda self: self._view("br_segs"))

    def __del__(self):
        try:
            lib().rksc_tables_free(C.byref(self.c))
        except Exception:
            pass


def rksc_tables_from_gate(branch_to_prefix, num_prefixes,
                          shared_off, shared_pages, shared_ntok,
                          priv_off, priv_pages, priv_ntok,
                          sfx_off, sfx_pages, sfx_ntok) -> Tables:
    """Host call: segment tables from a gate map (the library's result, wrapped without a copy)."""
    arrs = [_i32(a) for a in (branch_to_prefix, shared_off, shared_pages, shared_ntok,
                              priv_off, priv_pages, priv_ntok, sfx_off, sfx_pages, sfx_ntok)]
    out = _CTables()
    st = lib().rksc_tables_from_gate(len(arrs[0]), int(num_prefixes), *[_p(a) for a in arrs], C.byref(out))
    _check(st, "rksc_tables_from_gate")
    return LibTables(out)


class Plan:
    """Owner of an rksc_plan (destroyed with the object)."""

    def __init__(self, handle: int, layout: Layout, tables: Optional[Tables], num_branches: int):
        self._h = C.c_void_p(handle)
        self.layout = layout
        self.tables = tables      # None when the plan was created straight from a gate map
        self.num_branches = num_branches
        self._info = None

    def _query(self):
        if self._info is None:
            info = _CPlanInfo()
            _check(lib().rksc_plan_query(self._h, C.byref(info)), "rksc_plan_query")
            self._info = info
            self._mass_off = np.ctypeslib.as_array(info.mass_off, shape=(self.num_branches + 1,)).copy()
        return self._info

    workspace_bytes = property(lambda self: int(self._query().workspace_bytes))
    mass_elems = property(lambda self: int(self._query().mass_elems))
    num_work_items = property(lambda self: int(self._query().num_work_items))
    num_partial_rows = property(lambda self: int(self._query().num_partial_rows))
    unique_kv_tokens = property(lambda self: int(self._query().unique_kv_tokens))
    duplicated_kv_tokens = property(lambda self: int(self._query().duplicated_kv_tokens))
    on_device = property(lambda self: bool(self._query().on_device))
    num_pages_listed = property(lambda self: int(self._query().num_pages_listed))
    num_kernel_launches = property(lambda self: int(self._query().num_kernel_launches))

    @property
    def mass_off(self):
        self._query()
        return self._mass_off

    def item(self, i: int) -> np.ndarray:
        out = np.zeros(10, dtype=np.int32)
        _check(lib().rksc_plan_get_item(self._h, int(i), _p(out)), "rksc_plan_get_item")
        return out

    def items(self) -> np.ndarray:
        return np.stack([self.item(i) for i in range(self.num_work_items)]) if self.num_work_items else \
            np.zeros((0, 10), np.int32)

    def close(self):
        if self._h:
            lib().rksc_plan_destroy(self._h)
            self._h = C.c_void_p(None)

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def rksc_plan_create(layout, tables) -> Plan:
    lay = layout if isinstance(layout, Layout) else Layout.of(layout)
    tab = Tables.of(tables)
    h = C.c_void_p()
    _check(lib().rksc_plan_create(C.byref(lay.c), C.byref(tab.c), C.byref(h)), "rksc_plan_create")
    return Plan(h.value, lay, tab, tab.c.num_branches)


class GateLists:
    """The nine CSR arrays of the two-level page lists, marshalled once and reusable across steps."""

    def __init__(self, flat):
        self.num_prefixes = int(flat.num_prefixes)
        self.arrays = [_i32(getattr(flat, n)) for n in ("shared_off", "shared_pages", "shared_ntok", "priv_off",
                                                       "priv_pages", "priv_ntok", "sfx_off", "sfx_pages", "sfx_ntok")]
        self.ptrs = [_p(a) for a in self.arrays]


def rksc_plan_create_from_gate(layout, branch_to_prefix, lists) -> Plan:
    """rksc_tables_from_gate + rksc_plan_create in one host call (``lists``: a GateLists or an object with the CSR arrays)."""
    lay = layout if isinstance(layout, Layout) else Layout.of(layout)
    gl = lists if isinstance(lists, GateLists) else GateLists(lists)
    m = _i32(branch_to_prefix)
    h = C.c_void_p()
    _check(lib().rksc_plan_create_from_gate(C.byref(lay.c), len(m), gl.num_prefixes, _p(m), *gl.ptrs, C.byref(h)),
           "rksc_plan_create_from_gate")
    return Plan(h.value, lay, None, len(m))


def rksc_asks_gate(h_branch, h_root, cand_prefix, alpha: float, tau: float,
                   branch_to_prefix=None, sigma=None, stream=None):
    """Launches the gate kernel.  Returns (branch_to_prefix int32 [B], sigma fp32 [B]) on the device."""
    import torch
    assert h_branch.is_cuda and h_root.is_cuda and cand_prefix.is_cuda
    assert h_branch.dtype == torch.float32 and h_root.dtype == torch.float32 and cand_prefix.dtype == torch.int32
    assert h_branch.is_contiguous() and h_root.is_contiguous() and cand_prefix.is_contiguous()
    B, L, D = h_branch.shape
    P = h_root.shape[0]
    assert h_root.shape[1:] == (L, D) and cand_prefix.shape == (B,)
    if branch_to_prefix is None:
        branch_to_prefix = torch.empty(B, dtype=torch.int32, device=h_branch.device)
    if sigma is None:
        sigma = torch.empty(B, dtype=torch.float32, device=h_branch.device)
    st = lib().rksc_asks_gate(h_branch.data_ptr(), h_root.data_ptr(), cand_prefix.data_ptr(), B, P, L, D,
                              float(alpha), float(tau), branch_to_prefix.data_ptr(), sigma.data_ptr(),
                              _stream_ptr(stream, h_branch.device))
    _check(st, "rksc_asks_gate")
    return branch_to_prefix, sigma


def rksc_branch_decode_attention(plan: Plan, q, k_pool, v_pool, out=None, block_mass=None,
                                 workspace=None, device_status=None, stream=None, want_mass=True, phases=3):
    """Launches the attention.  Returns (out fp32 [B][Hq][d], block_mass fp32 flat or None, device_status).

    ``phases`` other than 3 goes through rksc_branch_decode_attention_phases (1 = segment kernel
    only, 2 = merge only), which exists so that events can be recorded between the launches."""
    import torch
    lay = plan.layout.c
    B = plan.num_branches
    assert q.is_cuda and q.dtype == torch.bfloat16 and q.is_contiguous()
    assert tuple(q.shape) == (B, lay.num_q_heads, lay.head_dim)
    for pool in (k_pool, v_pool):
        assert pool.is_cuda and pool.dtype == torch.bfloat16 and pool.is_contiguous()
        assert tuple(pool.shape) == (lay.num_pool_blocks, lay.num_kv_heads, 16, lay.head_dim)
    dev = q.device
    if out is None:
        out = torch.empty((B, lay.num_q_heads, lay.head_dim), dtype=torch.float32, device=dev)
    if block_mass is None and want_mass:
        block_mass = torch.empty(max(plan.mass_elems, 1), dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(plan.workspace_bytes, dtype=torch.uint8, device=dev)
    if device_status is None:
        device_status = torch.zeros(1, dtype=torch.int32, device=dev)
    args = (plan._h, q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(), out.data_ptr(),
            block_mass.data_ptr() if block_mass is not None else None,
            workspace.data_ptr(), workspace.numel() * workspace.element_size(),
            device_status.data_ptr(), _stream_ptr(stream, dev))
    if phases == 3:
        st = lib().rksc_branch_decode_attention(*args)
    else:
        st = lib().rksc_branch_decode_attention_phases(*args, int(phases))
    _check(st, "rksc_branch_decode_attention")
    return out, block_mass, device_status


def split_block_mass(plan: Plan, block_mass) -> list:
    """The flat block_mass buffer as one [Hq][nblk_b] host array per branch."""
    flat = block_mass.detach().cpu().numpy() if hasattr(block_mass, "detach") else np.asarray(block_mass)
    Hq = plan.layout.c.num_q_heads
    res = []
    for b in range(plan.num_branches):
        lo, hi = int(plan.mass_off[b]) * Hq, int(plan.mass_off[b + 1]) * Hq
        res.append(flat[lo:hi].reshape(Hq, -1) if hi > lo else np.zeros((Hq, 0), np.float32))
    return res


def rksc_branch_decode_attention_static(plan: Plan, q, k_pool, v_pool, out, block_mass, device_status, stream=None):
    """The attention for callers that may not allocate: no workspace argument, nothing is allocated here.

    Every buffer is the caller's (``out`` fp32 [B][Hq][d], ``block_mass`` fp32 flat or None,
    ``device_status`` int32 [1]); the partial results go to the scratch array compiled into the
    library.  Plans needing more than STATIC_WORKSPACE_BYTES raise RkscError (status -4).  Calls
    share that scratch, so keep them ordered on one stream per device."""
    st = lib().rksc_branch_decode_attention_static(
        plan._h, q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(), out.data_ptr(),
        block_mass.data_ptr() if block_mass is not None else None,
        device_status.data_ptr() if device_status is not None else None, _stream_ptr(stream, q.device))
    _check(st, "rksc_branch_decode_attention_static")
    return out, block_mass, device_status


def rksc_rsbcm_page_scores(plan: Plan, block_mass, score=None, stream=None):
    """RSBCM score of every table entry (Section 2.4): device fp64 [num_pages_listed] from the block
    masses the attention wrote for ``plan``."""
    import torch
    if score is None:
        score = torch.empty(plan.num_pages_listed, dtype=torch.float64, device=block_mass.device)
    st = lib().rksc_rsbcm_page_scores(plan._h, block_mass.data_ptr(), score.data_ptr(),
                                      _stream_ptr(stream, block_mass.device))
    _check(st, "rksc_rsbcm_page_scores")
    return score


def rksc_rsbcm_workspace_bytes(n: int) -> int:
    return int(lib().rksc_rsbcm_workspace_bytes(int(n)))


def rksc_rsbcm_evict(score, depth, capacity: int, evicted=None, num_evicted=None, workspace=None, stream=None):
    """Algorithm 4 on device arrays: marks the max(0, n - capacity) entries smallest by
    (score / (depth + 1), index).  Returns (evicted uint8 [n], num_evicted int32 [1])."""
    import torch
    n = int(score.numel())
    dev = score.device
    if evicted is None:
        evicted = torch.empty(n, dtype=torch.uint8, device=dev)
    if num_evicted is None:
        num_evicted = torch.empty(1, dtype=torch.int32, device=dev)
    if workspace is None:
        workspace = torch.empty(rksc_rsbcm_workspace_bytes(n), dtype=torch.uint8, device=dev)
    st = lib().rksc_rsbcm_evict(score.data_ptr(), depth.data_ptr(), n, int(capacity), evicted.data_ptr(),
                                num_evicted.data_ptr(), workspace.data_ptr(), workspace.numel(),
                                _stream_ptr(stream, dev))
    _check(st, "rksc_rsbcm_evict")
    return evicted, num_evicted


def rksc_tables_drop_evicted(tables, evicted) -> Tables:
    """Host call: the tables without the evicted entries (``evicted``: host uint8/bool [entries])."""
    t = Tables.of(tables)
    ev = np.ascontiguousarray(np.asarray(evicted).astype(np.uint8))
    out = _CTables()
    st = lib().rksc_tables_drop_evicted(C.byref(t.c), ev.ctypes.data_as(C.c_void_p), C.byref(out))
    _check(st, "rksc_tables_drop_evicted")
    return LibTables(out)


def rksc_tables_append_token(tables, new_pages):
    """Host call: one decode step on the tables.  Returns (Tables, page int32 [B], slot int32 [B])."""
    t = Tables.of(tables)
    B = int(t.c.num_branches)
    npg = _i32(new_pages) if new_pages is not None else None
    page = np.empty(max(B, 1), dtype=np.int32)
    slot = np.empty(max(B, 1), dtype=np.int32)
    out = _CTables()
    st = lib().rksc_tables_append_token(C.byref(t.c), _p(npg) if npg is not None else None, C.byref(out), _p(page), _p(slot))
    _check(st, "rksc_tables_append_token")
    return LibTables(out), page[:B], slot[:B]


def rksc_kv_append(layout, k_pool, v_pool, k_new, v_new, page, slot, stream=None):
    """Device call: the new token's keys and values (bf16 [B][Hkv][d]) into the paged pools at (page, slot)
    (device int32 [B])."""
    lay = layout if isinstance(layout, Layout) else Layout.of(layout)
    st = lib().rksc_kv_append(C.byref(lay.c), k_pool.data_ptr(), v_pool.data_ptr(), k_new.data_ptr(), v_new.data_ptr(),
                              int(k_new.shape[0]), page.data_ptr(), slot.data_ptr(), _stream_ptr(stream, k_pool.device))
    _check(st, "rksc_kv_append")


def rksc_cgee_logit_entropy(h, w_u, entropy=None, top1_prob=None, workspace=None, device_status=None, stream=None):
    """Entropy (nats) and top-1 probability of softmax(h W_u^T) per row of h (Section 2.3, Eq. 5 / Eq. 3).
    h bf16 [B][D], w_u bf16 [V][D] on the device.  Returns (entropy [B], top1_prob [B], device_status [1])."""
    import torch
    B, D = h.shape
    V = w_u.shape[0]
    dev = h.device
    if entropy is None:
        entropy = torch.empty(B, dtype=torch.float32, device=dev)
    if top1_prob is None:
        top1_prob = torch.empty(B, dtype=torch.float32, device=dev)
    if workspace is None:
        workspace = torch.empty(int(lib().rksc_cgee_workspace_bytes()), dtype=torch.uint8, device=dev)
    if device_status is None:
        device_status = torch.zeros(1, dtype=torch.int32, device=dev)
    st = lib().rksc_cgee_logit_entropy(h.data_ptr(), w_u.data_ptr(), B, D, V, entropy.data_ptr(), top1_prob.data_ptr(),
                                       workspace.data_ptr(), workspace.numel(), device_status.data_ptr(),
                                       _stream_ptr(stream, dev))
    _check(st, "rksc_cgee_logit_entropy")
    return entropy, top1_prob, device_status


def rksc_cgee_entropy_exit(entropy, entropy_prev, layer: int, l_min: int, theta: float, eps: float, exit_flags=None,
                           stream=None):
    """Algorithm 3's exit test per row (device fp32 arrays [B]); returns int32 flags [B]."""
    import torch
    B = int(entropy.numel())
    if exit_flags is None:
        exit_flags = torch.empty(B, dtype=torch.int32, device=entropy.device)
    st = lib().rksc_cgee_entropy_exit(entropy.data_ptr(), entropy_prev.data_ptr(), B, int(layer), int(l_min), float(theta),
                                      float(eps), exit_flags.data_ptr(), _stream_ptr(stream, entropy.device))
    _check(st, "rksc_cgee_entropy_exit")
    return exit_flags


def rksc_cgee_verify_skip(top1_per_step, tau_conf: float, r_gap: float, stream=None):
    """Level-1 gate (Eq. 3, 4): top1_per_step device fp32 [t][B] -> (confidence [B], skip int32 [1])."""
    import torch
    t, B = top1_per_step.shape
    dev = top1_per_step.device
    conf = torch.empty(B, dtype=torch.float32, device=dev)
    skip = torch.empty(1, dtype=torch.int32, device=dev)
    st = lib().rksc_cgee_verify_skip(top1_per_step.data_ptr(), t, B, float(tau_conf), float(r_gap), conf.data_ptr(),
                                     skip.data_ptr(), _stream_ptr(stream, dev))
    _check(st, "rksc_cgee_verify_skip")
    return conf, skip


def rksc_tables_for_suffix_prefill(tables, s: int) -> Tables:
    """Host call: tables of the B * s virtual branches whose decode attention is the suffix prefill of
    the last s tokens of every branch (see rksc_tables_for_suffix_prefill in rksc.h)."""
    t = Tables.of(tables)
    out = _CTables()
    st = lib().rksc_tables_for_suffix_prefill(C.byref(t.c), int(s), C.byref(out))
    _check(st, "rksc_tables_for_suffix_prefill")
    return LibTables(out)


def rksc_decode_step_host(layout, h_branch, h_root, cand_prefix, alpha, tau, flat, q, k_pool, v_pool,
                          branch_to_prefix, sigma, out, block_mass, mass_off=None, stream=None):
    """The whole path for host-resident per-step data (see rksc_decode_step_host in rksc.h).

    h_branch, h_root, q, branch_to_prefix, sigma, out, block_mass are HOST torch tensors (pinned for
    asynchronous copies); cand_prefix and the page lists (``flat``: an object with the nine CSR arrays
    and num_prefixes) are host int32 arrays; k_pool / v_pool are the device-resident pool.
    Returns the status word (0 = ok)."""
    lay = layout if isinstance(layout, Layout) else Layout.of(layout)
    B, L, D = h_branch.shape
    P = h_root.shape[0]
    cand = _i32(cand_prefix)
    lists = [_i32(getattr(flat, n)) for n in ("shared_off", "shared_pages", "shared_ntok", "priv_off", "priv_pages",
                                              "priv_ntok", "sfx_off", "sfx_pages", "sfx_ntok")]
    mo = None
    if mass_off is not None:
        assert mass_off.dtype == np.int64 and mass_off.shape[0] == B + 1
        mo = mass_off.ctypes.data
    st = lib().rksc_decode_step_host(
        C.byref(lay.c), h_branch.data_ptr(), h_root.data_ptr(), cand.ctypes.data, B, P, L, D, float(alpha), float(tau),
        *[_p(a) for a in lists], q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(),
        branch_to_prefix.data_ptr(), sigma.data_ptr() if sigma is not None else None, out.data_ptr(),
        block_mass.data_ptr() if block_mass is not None else None,
        block_mass.numel() if block_mass is not None else 0, mo, _stream_ptr(stream, k_pool.device))
    _check(st, "rksc_decode_step_host")
    return st


def rksc_debug_wait_timeout(limit_cycles: int, device_status, stream=None) -> int:
    """Self-test of the kernels' bounded wait (see rksc.h); returns the host status of the launch."""
    return int(lib().rksc_debug_wait_timeout(int(limit_cycles), device_status.data_ptr() if device_status is not None
                                             else None, _stream_ptr(stream, device_status.device if device_status
                                                                    is not None else None)))


class StepResult:
    """What rksc_pipeline_wait hands back for one step (host data)."""

    def __init__(self, status, branch_to_prefix, sigma, mass_off, info, segment_ms):
        self.status = status
        self.branch_to_prefix = branch_to_prefix
        self.sigma = sigma
        self.mass_off = mass_off
        self.mass_elems = int(info.mass_elems)
        self.workspace_bytes = int(info.workspace_bytes)
        self.num_work_items = int(info.num_work_items)
        self.num_kernel_launches = int(info.num_kernel_launches)
        self.unique_kv_tokens = int(info.unique_kv_tokens)
        self.num_pages_listed = int(info.num_pages_listed)
        self.segment_ms = segment_ms


class Pipeline:
    """rksc_pipeline_*: whole steps (gate, map to the host, tables + plan, attention) kept ``depth`` deep in
    flight by the library's own streams and host threads.  Argument marshalling only."""

    def __init__(self, layout, num_branches, hidden_shape, alpha, tau, lists, depth=4, mass_capacity=0, timing=0):
        lay = layout if isinstance(layout, Layout) else Layout.of(layout)
        gl = lists if isinstance(lists, GateLists) else GateLists(lists)
        L_, D = hidden_shape
        self.layout, self.B, self.depth = lay, int(num_branches), int(depth)
        h = C.c_void_p()
        _check(lib().rksc_pipeline_create(C.byref(lay.c), self.B, gl.num_prefixes, int(L_), int(D), float(alpha),
                                          float(tau), *gl.ptrs, int(depth), int(mass_capacity), int(timing),
                                          C.byref(h)), "rksc_pipeline_create")
        self._h = h.value
        self._keep = {}

    def submit(self, h_branch, h_root, cand_prefix, q, k_pool, v_pool, out, block_mass=None, after_stream=None) -> int:
        t = C.c_int64(-1)
        _check(lib().rksc_pipeline_submit(self._h, h_branch.data_ptr(), h_root.data_ptr(), cand_prefix.data_ptr(),
                                          q.data_ptr(), k_pool.data_ptr(), v_pool.data_ptr(), out.data_ptr(),
                                          block_mass.data_ptr() if block_mass is not None else None,
                                          _stream_ptr(after_stream, q.device) if after_stream is not None else None,
                                          C.byref(t)), "rksc_pipeline_submit")
        # the step reads these buffers until it has been waited for
        self._keep[t.value] = (h_branch, h_root, cand_prefix, q, k_pool, v_pool, out, block_mass)
        return int(t.value)

    def wait(self, ticket: int, check: bool = True) -> StepResult:
        m = np.empty(self.B, dtype=np.int32)
        sg = np.empty(self.B, dtype=np.float32)
        mo = np.zeros(self.B + 1, dtype=np.int64)
        info = _CPlanInfo()
        ms = C.c_float(0.0)
        st = lib().rksc_pipeline_wait(self._h, int(ticket), m.ctypes.data, sg.ctypes.data, mo.ctypes.data,
                                      C.byref(info), C.byref(ms))
        self._keep.pop(int(ticket), None)
        if check:
            _check(st, "rksc_pipeline_wait")
        return StepResult(int(st), m, sg, mo, info, float(ms.value))

    def close(self):
        if getattr(self, "_h", None):
            lib().rksc_pipeline_destroy(self._h)
            self._h = None
            self._keep.clear()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
