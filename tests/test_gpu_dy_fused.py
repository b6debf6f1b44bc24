"""The experts' backward that never writes dy_perm (mohge_row_tokens + mohge_expert_bwd_dy): the two
GEMMs that read dy_perm gather the rows of dy, the gate enters in the epilogue of the first, which
also writes gate * H for the second.  Against the oracle, and against the route through dy_perm."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import Workload, make_inputs

from _util import forced_switches, gpu_cfg, max_rel, oracle_layer, to_np64, tol_for

pytestmark = pytest.mark.gpu

CASES = [Workload("dyf_a", "bf16", 1000, 256, 3, 4, (352, 176, 88), 2, 4, seed=1),
         Workload("dyf_few", "bf16", 90, 256, 3, 4, (352, 176, 88), 2, 4, seed=2),
         Workload("dyf_odd_d", "bf16", 700, 200, 2, 4, (128, 72), 1, 2, seed=4),
         Workload("dyf_skew", "bf16", 1500, 256, 4, 8, (256, 192, 128, 64), 2, 6, zipf_beta=3.0, seed=5),
         Workload("dyf_wide", "bf16", 2100, 512, 2, 2, (512, 256), 2, 3, seed=6)]


def _run(wl, inp, logits32, dy_fused, accumulate=False):
    gcfg = gpu_cfg(wl)
    dev = {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in inp.items() if k not in ("w13", "w2")}
    w13, w2 = [w.cuda() for w in inp["w13"]], [w.cuda() for w in inp["w2"]]
    b = B.LayerBuffers(gcfg, wl.T)
    if dy_fused:
        b.dy_perm.fill_(float("nan"))                # the route must not depend on it
    lg = torch.from_numpy(np.ascontiguousarray(logits32)).cuda()
    B.layer_forward(gcfg, b, dev["x"], dev["w_router"], w13, w2, logit_bias=dev.get("logit_bias"),
                    logits_in=lg, aux=True)
    if accumulate:
        for g in range(wl.n_groups):
            b.dw13[g].fill_(1.0)
            b.dw2[g].fill_(-2.0)
    B.layer_backward(gcfg, b, dev["x"], dev["w_router"], w13, w2, dev["dy"], aux=True, dy_fused=dy_fused,
                     accumulate=accumulate)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    return b


@pytest.mark.parametrize("switch", ["", "MOHGE_TC_CG=1", "MOHGE_TC_CG=2,MOHGE_TC_WIDE=63", "MOHGE_TC_CG=2,MOHGE_TC_WIDE=0"])
@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
def test_backward_without_dy_perm_matches_the_oracle_and_the_route_through_dy_perm(wl, switch):
    inp = make_inputs(wl)
    fwd, bwd, logits32 = oracle_layer(wl, inp)
    with forced_switches(switch):
        f = _run(wl, inp, logits32, dy_fused=True)
        p = _run(wl, inp, logits32, dy_fused=False)
    tol = tol_for(wl.dtype)
    # the row map and the gate of every physical row
    dp = O.dispatch(fwd["expert_idx"], wl.n_experts, 128)
    tok = np.full(f.tok_of_prow.numel(), wl.T, np.int64)
    tok[dp["prow_of"].ravel()] = np.repeat(np.arange(wl.T), wl.k_experts)
    assert (f.tok_of_prow.cpu().numpy() == tok).all()
    rg = np.zeros(f.row_gate.numel(), np.float32)
    rg[dp["prow_of"].ravel()] = f.gate_w.cpu().numpy().ravel()
    assert np.array_equal(f.row_gate.cpu().numpy(), rg)
    # gate * H where rows exist (row r of h_saved times the gate of the row), to BF16 rounding
    for g in range(wl.n_groups):
        e0, e1 = g * wl.experts_per_group, (g + 1) * wl.experts_per_group
        sel = np.concatenate([np.arange(dp["aligned_offsets"][e], dp["aligned_offsets"][e] + dp["counts"][e])
                              for e in range(e0, e1)]).astype(np.int64)
        if sel.size:
            W = wl.group_width[g]
            got = to_np64(f.hs)[sel][:, :W]
            ref = to_np64(f.h)[sel][:, :W] * rg[sel, None]
            assert max_rel(got, ref) <= 1e-2
    # oracle parity of everything the two GEMMs feed
    assert max_rel(to_np64(f.dx), bwd["dx"]) <= tol
    assert max_rel(to_np64(f.dgate), bwd["dgate"]) <= tol
    assert max_rel(to_np64(f.dlogits), bwd["dlogits"]) <= tol
    for g in range(wl.n_groups):
        assert max_rel(to_np64(f.dw13[g]), bwd["dw13"][g]) <= tol
        assert max_rel(to_np64(f.dw2[g]), bwd["dw2"][g]) <= tol
    # and agreement with the route through dy_perm (other rounding places: tolerance, not bits)
    assert max_rel(to_np64(f.dx), to_np64(p.dx)) <= tol
    for g in range(wl.n_groups):
        assert max_rel(to_np64(f.dw2[g]), to_np64(p.dw2[g])) <= tol
        assert max_rel(to_np64(f.dw13[g]), to_np64(p.dw13[g])) <= tol


def test_backward_without_dy_perm_accumulates():
    wl = CASES[0]
    inp = make_inputs(wl)
    fwd, bwd, logits32 = oracle_layer(wl, inp)
    f = _run(wl, inp, logits32, dy_fused=True, accumulate=True)
    tol = tol_for(wl.dtype)
    for g in range(wl.n_groups):
        assert max_rel(to_np64(f.dw13[g]) - 1.0, bwd["dw13"][g]) <= tol
        assert max_rel(to_np64(f.dw2[g]) + 2.0, bwd["dw2"][g]) <= tol


def test_backward_without_dy_perm_with_a_gate_that_is_exactly_zero():
    """A selected expert whose gate is exactly zero: its rows get zero gradients, its gate gradient
    is still <dy, y_row> (the reduce kernel falls back to the definition)."""
    wl = Workload("dyf_zero_gate", "bf16", 600, 256, 2, 4, (128, 64), 2, 3, seed=12)
    inp = make_inputs(wl)
    gcfg = gpu_cfg(wl)
    dev = {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in inp.items() if k not in ("w13", "w2")}
    w13, w2 = [w.cuda() for w in inp["w13"]], [w.cuda() for w in inp["w2"]]

    def run(dy_fused):
        b = B.LayerBuffers(gcfg, wl.T)
        B.layer_forward(gcfg, b, dev["x"], dev["w_router"], w13, w2, logit_bias=dev.get("logit_bias"), aux=True)
        b.gate_w[::7, 1] = 0.0                       # after the forward: the backward sees zero gates
        B.layer_backward(gcfg, b, dev["x"], dev["w_router"], w13, w2, dev["dy"], aux=True, dy_fused=dy_fused)
        torch.cuda.synchronize()
        assert B.mohge_get_device_status(b.ws) == 0
        return b

    f, p = run(True), run(False)
    tol = tol_for(wl.dtype)
    assert float(f.dgate[::7, 1].abs().max()) > 0
    assert max_rel(to_np64(f.dgate), to_np64(p.dgate)) <= tol
    assert max_rel(to_np64(f.dx), to_np64(p.dx)) <= tol
    for g in range(wl.n_groups):
        assert max_rel(to_np64(f.dw2[g]), to_np64(p.dw2[g])) <= tol


def test_backward_without_dy_perm_at_the_slice_of_the_large_workload():
    """Tile forms and contraction lengths of the large workload (double-width CTA-pair entries,
    K = 4096): the route without dy_perm against the route through it, on the device."""
    from paper_2604_23108_b200.inputs import WORKLOADS, make_device_inputs
    wl = WORKLOADS["cfg5_slice"]
    dev = torch.device("cuda", 0)
    gcfg = gpu_cfg(wl)
    inp = make_device_inputs(wl, dev)
    res = []
    for dy_fused in (False, True):
        b = B.LayerBuffers(gcfg, wl.T, device=dev)
        B.layer_forward(gcfg, b, inp["x"], inp["w_router"], inp["w13"], inp["w2"], logit_bias=inp["logit_bias"], aux=True)
        B.layer_backward(gcfg, b, inp["x"], inp["w_router"], inp["w13"], inp["w2"], inp["dy"], aux=True, dy_fused=dy_fused)
        torch.cuda.synchronize()
        assert B.mohge_get_device_status(b.ws) == 0
        res.append(b)
    p, f = res
    rel = lambda a, c: float((a.float() - c.float()).abs().max() / c.float().abs().max())
    tol = tol_for(wl.dtype)
    assert torch.equal(p.expert_idx, f.expert_idx)
    assert rel(f.dx, p.dx) <= tol and rel(f.dgate, p.dgate) <= tol and rel(f.dw_router, p.dw_router) <= tol
    for g in range(wl.n_groups):
        for i in range(wl.experts_per_group):
            assert rel(f.dw2[g][i], p.dw2[g][i]) <= tol, (g, i)
            assert rel(f.dw13[g][i], p.dw13[g][i]) <= tol, (g, i)
