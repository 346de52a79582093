"""The bounded wait every kernel of the library relies on, made to run out on purpose.

rksc_debug_wait_timeout launches a CTA whose warps wait, with a limit of a few hundred thousand SM
cycles, on a barrier that nothing completes.  The wait gives up, records RKSC_ERR_DEVICE_TIMEOUT in
the status word and the kernel returns: no trap, no hang, the context stays usable (checked by a
normal attention call right after).  Nothing here faults the device."""
import numpy as np
import pytest

import workloads
from helpers import check_attention, oracle_attention


def test_arguments_are_checked_on_the_host():
    import paper_2606_09937_b200 as rk
    assert rk.lib().rksc_debug_wait_timeout(0, None, None) == -1
    assert rk.lib().rksc_debug_wait_timeout(1 << 40, None, None) == -1
    assert rk.lib().rksc_debug_wait_timeout(1000, None, None) == -1     # no status word


@pytest.mark.gpu
def test_wait_runs_out_sets_the_status_and_leaves_the_context_usable():
    import time
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    t0 = time.perf_counter()
    assert rk.rksc_debug_wait_timeout(400_000, status) == 0          # about 0.2 ms at 2 GHz
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 5.0
    assert int(status.item()) == -6                                   # RKSC_ERR_DEVICE_TIMEOUT
    assert rk.rksc_strerror(-6)
    # the device is fine: a normal call afterwards matches the oracle
    w = workloads.make_config("tiny")
    plan = rk.rksc_plan_create(w.layout, w.tables)
    out, mass, st = rk.rksc_branch_decode_attention(plan, w.q.to(dev), w.k_pool.to(dev), w.v_pool.to(dev))
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ref_out, ref_m = oracle_attention(w)
    check_attention(out.cpu().numpy(), rk.split_block_mass(plan, mass), ref_out, ref_m)
