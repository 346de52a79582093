"""B200 (sm_100a) ASKS hot path: similarity gate + shared-prefix branch-decode attention.

The work is done by hand-written CUDA kernels behind a C ABI (``include/rksc.h``,
built into ``librksc.so`` in this directory).  This package is a thin ctypes
binding with the same entry-point names; torch is used for device memory and
streams only.  There is no CPU or eager fallback: if the library cannot be
loaded, importing the binding's functions raises.
"""
from .binding import (  # noqa: F401
    RkscError,
    Layout,
    Tables,
    Plan,
    lib,
    lib_path,
    rksc_strerror,
    rksc_asks_gate,
    rksc_tables_from_gate,
    rksc_plan_create,
    rksc_plan_create_from_gate,
    GateLists,
    rksc_branch_decode_attention,
    rksc_branch_decode_attention_static,
    rksc_decode_step_host,
    rksc_rsbcm_page_scores,
    rksc_rsbcm_workspace_bytes,
    rksc_rsbcm_evict,
    rksc_tables_drop_evicted,
    rksc_tables_for_suffix_prefill,
    rksc_tables_append_token,
    rksc_kv_append,
    rksc_cgee_logit_entropy,
    rksc_cgee_entropy_exit,
    rksc_cgee_verify_skip,
    rksc_debug_wait_timeout,
    Pipeline,
    StepResult,
    STATIC_WORKSPACE_BYTES,
    split_block_mass,
    EXPORTED_SYMBOLS,
)
