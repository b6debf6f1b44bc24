"""GPU parity of the layer WITH shared experts: routed sum + one ungated dense SwiGLU FFN over
every token (N_s experts concatenated along the hidden axis), forward and backward, against the
oracle.  The shared FFN runs on the grouped-expert kernels with x as a single segment, so the
cases use token counts that are not multiples of the 128/256-row tiles."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import Workload, make_inputs, make_shared_weights

from _util import gpu_cfg, max_rel, oracle_cfg, to_np64, tol_for

pytestmark = pytest.mark.gpu

CASES = [
    (Workload("sh_f32", "f32", 333, 72, 3, 3, (40, 24, 56), 2, 4, seed=3), 48),
    (Workload("sh_bf16", "bf16", 1000, 256, 3, 4, (352, 176, 88), 2, 4, seed=1), 2 * 176),
    (Workload("sh_bf16_wide", "bf16", 777, 512, 4, 8, (384, 256, 192, 128), 2, 6, seed=2), 2 * 384),
    (Workload("sh_bf16_one_tile", "bf16", 100, 128, 2, 4, (64, 32), 1, 2, seed=5), 64),
]


@pytest.mark.parametrize("wl,Ws", CASES, ids=[c[0].name for c in CASES])
def test_layer_with_shared_experts(wl, Ws):
    inp = make_inputs(wl)
    w13_s, w2_s = make_shared_weights(wl, Ws)
    ocfg = oracle_cfg(wl)
    x64, wr64 = to_np64(inp["x"]), to_np64(inp["w_router"])
    w13 = [to_np64(w) for w in inp["w13"]]
    w2 = [to_np64(w) for w in inp["w2"]]
    sh = (to_np64(w13_s), to_np64(w2_s))
    logits32 = O.router_logits(x64, wr64).astype(np.float32)
    fwd = O.layer_forward(ocfg, x64, wr64, w13, w2, logits=logits32.astype(np.float64), mode="spec", shared=sh)
    bwd = O.layer_backward(fwd, w13, w2, to_np64(inp["dy"]), with_aux=True, shared=sh)

    gcfg = gpu_cfg(wl)
    T = wl.T
    b = B.LayerBuffers(gcfg, T, shared_width=Ws)
    dev = {k: v.cuda() for k, v in inp.items() if isinstance(v, torch.Tensor)}
    dw13, dw2 = [w.cuda() for w in inp["w13"]], [w.cuda() for w in inp["w2"]]
    shd = (w13_s.cuda(), w2_s.cuda())
    lg = torch.from_numpy(logits32).cuda()
    for rep in range(2):                      # the second pass reuses every buffer
        B.layer_forward(gcfg, b, dev["x"], dev["w_router"], dw13, dw2, logits_in=lg, shared=shd)
        B.layer_backward(gcfg, b, dev["x"], dev["w_router"], dw13, dw2, dev["dy"], shared=shd)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    tol = tol_for(wl.dtype)
    assert (b.expert_idx.cpu().numpy() == fwd["expert_idx"]).all()
    c = fwd["shared"]
    au = to_np64(b.au_sh)
    assert max_rel(au[:, :Ws], c["A"]) <= tol and max_rel(au[:, Ws:], c["U"]) <= tol
    assert max_rel(to_np64(b.h_sh), c["H"]) <= tol
    assert max_rel(to_np64(b.y_sh), c["Y"]) <= tol
    assert max_rel(to_np64(b.y), fwd["y"]) <= tol
    sb = bwd["shared"]
    dau = to_np64(b.dau_sh)
    assert max_rel(dau[:, :Ws], sb["dA"]) <= tol and max_rel(dau[:, Ws:], sb["dU"]) <= tol
    assert max_rel(to_np64(b.dx_sh), sb["dx"]) <= tol
    assert max_rel(to_np64(b.dw13_sh), sb["dw13"]) <= tol
    assert max_rel(to_np64(b.dw2_sh), sb["dw2"]) <= tol
    assert max_rel(to_np64(b.dx), bwd["dx"]) <= tol
    for g in range(wl.n_groups):              # the routed experts are untouched by the addition
        assert max_rel(to_np64(b.dw13[g]), bwd["dw13"][g]) <= tol
        assert max_rel(to_np64(b.dw2[g]), bwd["dw2"][g]) <= tol
    # accumulate adds into the shared weight gradients
    ref13, ref2 = b.dw13_sh.clone(), b.dw2_sh.clone()
    B.mohge_shared_bwd(gcfg, T, Ws, dev["dy"], dev["x"], b.au_sh, b.h_sh, shd[0], shd[1], b.dau_sh,
                       b.dx_sh, b.dw13_sh, b.dw2_sh, 1, b.ws)
    torch.cuda.synchronize()
    assert max_rel(to_np64(b.dw13_sh), 2 * to_np64(ref13)) <= 1e-6
    assert max_rel(to_np64(b.dw2_sh), 2 * to_np64(ref2)) <= 1e-6


def test_shared_width_is_validated():
    wl = CASES[1][0]
    gcfg = gpu_cfg(wl)
    b = B.LayerBuffers(gcfg, wl.T, shared_width=64)
    x = torch.zeros(wl.T, wl.d_model, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(B.MohgeError):
        B.mohge_shared_fwd(gcfg, wl.T, 60, x, b.dw13_sh, b.dw2_sh, b.au_sh, b.h_sh, b.y_sh, b.ws)


def test_paper_shaped_layer_with_two_shared_experts_at_full_size():
    """The paper's 3B-scale layer (eight groups, K_g = 3, K_e = 6, 16384 tokens) with N_s = 2
    shared experts of the baseline's width 1024, every element against the oracle."""
    from paper_2604_23108_b200.inputs import WORKLOADS, make_device_inputs
    wl = WORKLOADS["paper_3b_layer"]
    Ws = 2 * 1024
    dev = torch.device("cuda", 0)
    inp = make_device_inputs(wl, dev)
    shd = make_shared_weights(wl, Ws, device=dev)
    gcfg = gpu_cfg(wl)
    b = B.LayerBuffers(gcfg, wl.T, device=dev, shared_width=Ws)
    B.layer_forward(gcfg, b, inp["x"], inp["w_router"], inp["w13"], inp["w2"], shared=shd)
    B.layer_backward(gcfg, b, inp["x"], inp["w_router"], inp["w13"], inp["w2"], inp["dy"], shared=shd)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    logits32 = b.logits.cpu().numpy()
    w13 = [to_np64(w) for w in inp["w13"]]
    w2 = [to_np64(w) for w in inp["w2"]]
    sh = (to_np64(shd[0]), to_np64(shd[1]))
    fwd = O.layer_forward(oracle_cfg(wl), to_np64(inp["x"]), to_np64(inp["w_router"]), w13, w2,
                          logits=logits32.astype(np.float64), mode="spec", shared=sh)
    bwd = O.layer_backward(fwd, w13, w2, to_np64(inp["dy"]), with_aux=True, shared=sh)
    tol = 2e-2
    assert (b.expert_idx.cpu().numpy() == fwd["expert_idx"]).all()
    assert max_rel(to_np64(b.y_sh), fwd["shared"]["Y"]) <= tol
    assert max_rel(to_np64(b.y), fwd["y"]) <= tol
    assert max_rel(to_np64(b.dx), bwd["dx"]) <= tol
    assert max_rel(to_np64(b.dw13_sh), bwd["shared"]["dw13"]) <= tol
    assert max_rel(to_np64(b.dw2_sh), bwd["shared"]["dw2"]) <= tol
