"""CPU oracle for the ASKS gate and branch-decode attention (fp64, numpy).

TEST INFRASTRUCTURE, NOT A PRODUCT PATH.  Only the test-suite, the smoke check
and the benchmark's CPU-baseline leg may import this package.  It shares no
code with the CUDA library and imports nothing from it; the CUDA package
imports nothing from here.

Every function is the plain definition of what the paper's method computes,
written for reading rather than speed:

* ``asks_gate``        - Eq. 2 and Algorithm 2 (layer-weighted cosine, threshold).
* ``tables_from_gate`` - the block tables that replace Algorithm 1's broadcast
                         copy of the prefix cache (line 3).
* ``branch_decode_attention`` - scaled-dot-product attention of one decode query
                         per (branch, head) over a physically duplicated
                         prefix + suffix (the paper's repeat_interleave + clone,
                         Section 2.2 "KV broadcast and batched decode"), plus the
                         softmax mass per KV block.
* ``page_scores`` / ``rsbcm_evict`` - the eviction that consumes those masses
                         (Section 2.4, Algorithm 4).
* ``suffix_prefill_attention`` / ``suffix_prefill_tables`` - the s suffix tokens of
                         every branch attending causally on top of the shared cache
                         (Appendix "Stepwise Batched Decode", step 1), and the tables
                         that express it as a decode attention over B * s virtual branches.

* ``logit_entropy`` / ``entropy_exit`` / ``generation_confidence`` / ``verify_skip`` - the
                         numerics of CGEE (Section 2.3, Eq. 3-5, Algorithm 3).
* ``append_token`` / ``write_token`` - one step of the token-by-token decode on the paged
                         cache (Appendix "Stepwise Batched Decode", step 2): index work.

Parity pins: every function here is pinned by the CPU tests against closed
forms, brute force on tiny inputs and invariants; none is "parity unpinned".
"""
from .asks_gate import layer_weights, asks_gate, layer_cosines  # noqa: F401
from .block_tables import (  # noqa: F401
    tables_from_gate,
    segment_sharers,
    logical_block_counts,
    mass_offsets,
)
from .branch_attention import branch_decode_attention, to_f32_numpy  # noqa: F401
from .rsbcm import page_scores, rsbcm_evict, apply_eviction  # noqa: F401
from .suffix_prefill import suffix_prefill_attention, suffix_prefill_tables  # noqa: F401
from .cgee import logit_entropy, entropy_exit, generation_confidence, verify_skip  # noqa: F401
from .decode_loop import append_token, write_token  # noqa: F401
