"""Seeded synthetic inputs for the ASKS gate and branch-decode attention.

This package only *draws and arranges* inputs (random tensors, page ids, token
counts, segment lists).  It holds none of the method's arithmetic: no cosine,
no softmax, no table construction from a gate map.  Both the CUDA path's tests
and the CPU oracle's tests take their inputs from here; neither the oracle nor
the CUDA package is imported.
"""
from .generators import (  # noqa: F401
    BLOCK,
    Layout,
    Tables,
    FlatLists,
    GateInputs,
    Workload,
    make_from_segments,
    make_gate_inputs,
    make_config,
    make_tiny,
    make_tiny_gate_tables,
    make_qwen_layer,
    make_tot,
    make_batched_serving,
    make_long_context,
    make_diverse_phrasing,
    punch_holes,
    lowest_mass_pages,
    make_block_masses,
    make_eviction_inputs,
    make_cgee_inputs,
    layer_variant,
    unique_kv_bytes,
    duplicated_kv_bytes,
    CONFIG_NAMES,
)
