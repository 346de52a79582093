"""The layers of one decode step captured in a CUDA graph (Appendix "Stepwise Batched Decode": every
layer of the step attends through the same tables, so one plan serves all of them).

The attention entry points only enqueue work on the caller's stream - no allocation, no
synchronisation, no host read-back - so a caller may record the calls of all L layers into one
graph and replay it.  These tests capture L calls (one plan, one workspace, a pool and an output
per layer), replay the graph, and compare every layer with the fp64 oracle; a second replay after
the queries were overwritten in place checks that the graph reads its inputs at replay time.
"""
import dataclasses

import numpy as np
import pytest

import workloads
from helpers import oracle_attention, check_attention

pytestmark = pytest.mark.gpu


def _capture_layers(rk, torch, plan, layers, dev, static):
    B, Hq, d = layers[0]["q"].shape
    ws = torch.empty(max(plan.workspace_bytes, 256), dtype=torch.uint8, device=dev)
    status = torch.zeros(1, dtype=torch.int32, device=dev)
    for lay in layers:
        lay["out"] = torch.full((B, Hq, d), float("nan"), dtype=torch.float32, device=dev)
        lay["mass"] = torch.full((max(plan.mass_elems, 1),), float("nan"), dtype=torch.float32, device=dev)

    def enqueue():
        for lay in layers:
            if static:
                rk.rksc_branch_decode_attention_static(plan, lay["q"], lay["k"], lay["v"], lay["out"], lay["mass"],
                                                       status)
            else:
                rk.rksc_branch_decode_attention(plan, lay["q"], lay["k"], lay["v"], out=lay["out"],
                                                block_mass=lay["mass"], workspace=ws, device_status=status)

    # one eager pass first: lazy one-time set-up (function attributes) stays out of the capture
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        enqueue()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    for lay in layers:
        lay["out"].fill_(float("nan"))
        lay["mass"].fill_(float("nan"))
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        enqueue()
    return graph, status


@pytest.mark.parametrize("static", [False, True], ids=["caller_workspace", "built_in_scratch"])
def test_three_layers_in_one_graph_match_the_oracle_on_every_replay(static):
    import torch
    import paper_2606_09937_b200 as rk

    dev = torch.device("cuda:0")
    # a prefix shared by six branches (tensor-core items), one shared by two, private suffixes with
    # ragged last pages (warp items): all three kernels are in the graph
    seg_ntok = [900, 77] + [33 + 5 * b for b in range(6)]
    br = [[0, 1, 2 + b] if b < 2 else [0, 2 + b] for b in range(6)]
    w0 = workloads.make_from_segments("layers", 28, 4, 128, seg_ntok, br, seed=91)
    ws_host = [workloads.layer_variant(w0, l) for l in range(3)]
    plan = rk.rksc_plan_create(w0.layout, w0.tables)
    layers = [dict(q=w.q.to(dev).clone(), k=w.k_pool.to(dev), v=w.v_pool.to(dev)) for w in ws_host]
    graph, status = _capture_layers(rk, torch, plan, layers, dev, static)

    for replay in range(2):
        if replay == 1:
            # new queries written into the captured buffers: the next replay must use them
            ws_host = [dataclasses.replace(ws_host[l], q=workloads.layer_variant(w0, l + 3).q) for l in range(3)]
            for lay, w in zip(layers, ws_host):
                lay["q"].copy_(w.q.to(dev))
        graph.replay()
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        for lay, w in zip(layers, ws_host):
            ref_out, ref_mass = oracle_attention(w)
            check_attention(lay["out"].cpu().numpy(), rk.split_block_mass(plan, lay["mass"]), ref_out, ref_mass)
    # the layers really differ (a graph that ran one layer three times would not pass the above,
    # and this guards the guard)
    assert not np.allclose(layers[0]["out"].cpu().numpy(), layers[1]["out"].cpu().numpy(), atol=1e-2)
