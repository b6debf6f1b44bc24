"""The entry points that never write x_perm (mohge_dispatch_indices, mohge_expert_fwd_gather,
mohge_expert_bwd_gather): the two GEMMs that read x_perm gather the rows of x through TMA.  They
must give the oracle's results and, tile for tile, the bits of the route through x_perm."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import Workload, make_inputs

from _util import forced_switches, gpu_cfg, max_rel, oracle_layer, to_np64, tol_for

pytestmark = pytest.mark.gpu

CASES = [Workload("gather_a", "bf16", 1000, 256, 3, 4, (352, 176, 88), 2, 4, seed=1),
         Workload("gather_few", "bf16", 90, 256, 3, 4, (352, 176, 88), 2, 4, seed=2),
         Workload("gather_odd_d", "bf16", 700, 200, 2, 4, (128, 72), 1, 2, seed=4),
         Workload("gather_skew", "bf16", 1500, 256, 4, 8, (256, 192, 128, 64), 2, 6, zipf_beta=3.0, seed=5)]


def _run(wl, inp, logits32, gather):
    gcfg = gpu_cfg(wl)
    dev = {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in inp.items() if k not in ("w13", "w2")}
    w13, w2 = [w.cuda() for w in inp["w13"]], [w.cuda() for w in inp["w2"]]
    b = B.LayerBuffers(gcfg, wl.T)
    b.x_perm.fill_(float("nan"))                     # the gathering route must not depend on it
    lg = torch.from_numpy(np.ascontiguousarray(logits32)).cuda()
    B.layer_forward(gcfg, b, dev["x"], dev["w_router"], w13, w2, logit_bias=dev.get("logit_bias"),
                    logits_in=lg, aux=True, gather=gather)
    B.layer_backward(gcfg, b, dev["x"], dev["w_router"], w13, w2, dev["dy"], aux=True, gather=gather)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    return b


@pytest.mark.parametrize("switch", ["", "MOHGE_TC_CG=1", "MOHGE_TC_CG=2,MOHGE_TC_WIDE=63", "MOHGE_TC_CG=2,MOHGE_TC_WIDE=0"])
@pytest.mark.parametrize("wl", CASES, ids=lambda w: w.name)
def test_gathering_route_matches_the_oracle_and_the_route_through_x_perm(wl, switch):
    inp = make_inputs(wl)
    fwd, bwd, logits32 = oracle_layer(wl, inp)
    with forced_switches(switch):
        g = _run(wl, inp, logits32, gather=True)
        p = _run(wl, inp, logits32, gather=False)
    tol = tol_for(wl.dtype)
    # the row map: token of every occupied physical row, T elsewhere
    dp = O.dispatch(fwd["expert_idx"], wl.n_experts, 128)
    tok = np.full(g.tok_of_prow.numel(), wl.T, np.int64)
    tok[dp["prow_of"].ravel()] = np.repeat(np.arange(wl.T), wl.k_experts)
    assert (g.tok_of_prow.cpu().numpy() == tok).all()
    for name in ("counts", "row_of", "prow_of", "src_of"):
        assert torch.equal(getattr(g, name), getattr(p, name)), name
    # oracle parity of what the two gathering GEMMs feed
    assert max_rel(to_np64(g.y), fwd["y"]) <= tol
    assert max_rel(to_np64(g.dx), bwd["dx"]) <= tol
    for grp in range(wl.n_groups):
        assert max_rel(to_np64(g.dw13[grp]), bwd["dw13"][grp]) <= tol
        assert max_rel(to_np64(g.dw2[grp]), bwd["dw2"][grp]) <= tol
    # and the same bits as the route through x_perm
    bits = lambda t: t.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32)
    used = int(dp["aligned_offsets"][-1])            # rows past the last segment are never written
    for name in ("y", "dx", "dgate", "dw_router"):
        assert torch.equal(bits(getattr(g, name)), bits(getattr(p, name))), name
    for name in ("y_perm", "dx_perm"):
        assert torch.equal(bits(getattr(g, name)[:used]), bits(getattr(p, name)[:used])), name
    for grp in range(wl.n_groups):
        assert torch.equal(g.dw13[grp], p.dw13[grp]) and torch.equal(g.dw2[grp], p.dw2[grp])


def test_gathering_entry_points_refuse_the_fp32_path():
    wl = Workload("gather_f32", "f32", 64, 32, 2, 4, (32, 16), 1, 2)
    gcfg = gpu_cfg(wl)
    b = B.LayerBuffers(gcfg, wl.T)
    x = torch.zeros(wl.T, wl.d_model, device="cuda")
    w13 = [torch.zeros(4, 2 * w, 32, device="cuda") for w in wl.group_width]
    w2 = [torch.zeros(4, 32, w, device="cuda") for w in wl.group_width]
    with pytest.raises(B.MohgeError, match="BF16"):
        B.mohge_expert_fwd_gather(gcfg, wl.T, x, b.tok_of_prow, b.counts, b.aligned, w13, w2, b.au, b.h,
                                  b.y_perm, b.ws)
