"""The layer step under CUDA graph capture.

Every launch of the path takes its sizes from the configuration and the token count; what depends
on the batch (counts, offsets, tile lists, statistics) stays in device memory.  So one captured
step must serve every later batch of the same T that is written into the same buffers: a replay
on a new batch is compared, bit for bit, with stream launches on that batch, and its forward
output with the oracle.
"""
import numpy as np
import pytest
import torch

from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import Workload, make_inputs

from _util import gpu_cfg, max_rel, oracle_layer, to_np64, tol_for

pytestmark = pytest.mark.gpu

OUTPUTS = ("logits", "expert_idx", "gate_w", "counts", "prow_of", "y", "dx", "dgate", "dlogits",
           "dw_router", "loss")


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_captured_step_replays_on_a_new_batch(dtype):
    wl_a = Workload("graph_a", dtype, 777, 128, 3, 4, (192, 64, 136), 2, 4, seed=31)
    wl_b = Workload("graph_b", dtype, 777, 128, 3, 4, (192, 64, 136), 2, 4, seed=32)
    inp_a, inp_b = make_inputs(wl_a), make_inputs(wl_b)
    gcfg = gpu_cfg(wl_a)
    x, dy = inp_a["x"].cuda(), inp_a["dy"].cuda()
    w_r = inp_a["w_router"].cuda()
    w13 = [w.cuda() for w in inp_a["w13"]]
    w2 = [w.cuda() for w in inp_a["w2"]]
    b = B.LayerBuffers(gcfg, wl_a.T)

    def step():
        B.layer_forward(gcfg, b, x, w_r, w13, w2, aux=True)
        B.layer_backward(gcfg, b, x, w_r, w13, w2, dy, aux=True)

    side = torch.cuda.Stream()                       # warm-up on a side stream, as capture wants
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()
    torch.cuda.current_stream().wait_stream(side)
    n0 = B.mohge_launch_count()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    assert B.mohge_launch_count() - n0 > 0           # the capture went through this library

    # a new batch (other tokens, other routing, other expert loads) into the captured buffers
    x.copy_(inp_b["x"].cuda())
    dy.copy_(inp_b["dy"].cuda())
    graph.replay()
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    got = {k: getattr(b, k).clone() for k in OUTPUTS}
    got_dw13 = [t.clone() for t in b.dw13]
    got_dw2 = [t.clone() for t in b.dw2]

    step()                                           # the same batch by stream launches
    torch.cuda.synchronize()
    for k in OUTPUTS:
        assert torch.equal(got[k], getattr(b, k)), k
    for g in range(wl_a.n_groups):
        assert torch.equal(got_dw13[g], b.dw13[g]) and torch.equal(got_dw2[g], b.dw2[g])

    inp_b = dict(inp_b, w_router=inp_a["w_router"], w13=inp_a["w13"], w2=inp_a["w2"])
    fwd, bwd, _ = oracle_layer(wl_b, inp_b, logits32=got["logits"].cpu().numpy())
    assert (got["expert_idx"].cpu().numpy() == fwd["expert_idx"]).all()
    assert max_rel(to_np64(got["y"]), fwd["y"]) <= tol_for(dtype)
    assert max_rel(to_np64(got["dx"]), bwd["dx"]) <= tol_for(dtype)
    assert not np.array_equal(fwd["expert_idx"],
                              oracle_layer(wl_a, inp_a)[0]["expert_idx"])   # the batches do differ
