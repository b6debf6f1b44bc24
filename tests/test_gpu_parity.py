"""GPU parity: every C-ABI step against the fp64 oracle, element by element, on seeded inputs.

Bars: routing indices, per-expert counts and the permutation are bit-exact given identical
router logits; float outputs and gradients within max|a-b|/max|b| <= 1e-5 (FP32 layer) or
2e-2 (BF16 in, FP32 accumulate).
"""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import WORKLOADS, Workload, make_inputs

from _util import forced_switches, gpu_cfg, gpu_layer, max_rel, oracle_cfg, oracle_layer, to_np64, tol_for

pytestmark = pytest.mark.gpu

# small cases the oracle finishes in seconds; they span several 128-row tiles, 256-token
# dispatch chunks and ragged tails, odd widths (88, 176, 352) and non-power-of-two N
CASES = {
    "cfg1": WORKLOADS["cfg1_tiny_f32"],
    "f32_ragged": Workload("f32_ragged", "f32", 333, 72, 3, 3, (40, 24, 56), 2, 4, seed=3),
    "bf16_small": Workload("bf16_small", "bf16", 1000, 256, 3, 4, (352, 176, 88), 2, 4, seed=1),
    "bf16_wide": Workload("bf16_wide", "bf16", 777, 512, 4, 8, (384, 256, 192, 128), 2, 6, seed=2),
    "bf16_paper_shape": Workload("bf16_paper_shape", "bf16", 600, 256, 8, 4,
                                 (64, 80, 96, 128, 160, 192, 208, 224), 3, 6, seed=4),
    "bf16_odd_d": Workload("bf16_odd_d", "bf16", 500, 200, 2, 4, (72, 40), 1, 3, seed=6),
    # few tokens: split-K router logits (3 row tiles, 8 k-blocks) and, at 100 rows per expert,
    # the single-CTA form of the grouped GEMMs
    "bf16_few_tokens": Workload("bf16_few_tokens", "bf16", 300, 512, 3, 4, (256, 128, 64), 2, 4, seed=7),
    "bf16_skew": Workload("bf16_skew", "bf16", 1500, 256, 4, 8, (256, 192, 128, 64), 2, 6,
                          zipf_beta=3.0, seed=5),
}


@pytest.fixture(scope="module", params=list(CASES))
def case(request):
    wl = CASES[request.param]
    inp = make_inputs(wl)
    fwd, bwd, logits32 = oracle_layer(wl, inp)
    b, dev = gpu_layer(wl, inp, logits32=logits32)
    return wl, inp, fwd, bwd, logits32, b, dev


def test_router_logits_match(case):
    wl, inp, fwd, bwd, logits32, b, dev = case
    gcfg = gpu_cfg(wl)
    T = inp["x"].shape[0]
    b2 = B.LayerBuffers(gcfg, T)
    B.mohge_route(gcfg, T, dev["x"], dev["w_router"], dev.get("logit_bias"), None, b2.logits,
                  b2.group_idx, b2.expert_idx, b2.gate_w, b2.gs, b2.esp, b2.ws)
    torch.cuda.synchronize()
    ref = fwd["logits"]
    assert max_rel(to_np64(b2.logits), ref) <= 1e-5
    # selections from the GPU's own logits agree wherever the fp64 margins are not razor thin
    d = O.route_definition(oracle_cfg(wl), ref)
    GS = np.sort(d["GS"], axis=1)[:, ::-1]
    ok = np.ones(T, bool)
    if wl.k_groups < wl.n_groups:
        ok &= (GS[:, wl.k_groups - 1] - GS[:, wl.k_groups]) / GS[:, wl.k_groups - 1] > 1e-3
    keys = np.sort(np.where(np.repeat(d["group_mask"], wl.experts_per_group, 1), d["ESpp"], -1.0),
                   axis=1)[:, ::-1]
    if wl.k_experts < wl.k_groups * wl.experts_per_group:
        ok &= (keys[:, wl.k_experts - 1] - keys[:, wl.k_experts]) / keys[:, wl.k_experts - 1] > 1e-3
    assert ok.mean() > 0.9
    gi = b2.group_idx.cpu().numpy()
    ei = b2.expert_idx.cpu().numpy()
    assert (np.sort(gi[ok], 1) == np.sort(d["group_idx"][ok], 1)).all()
    assert (np.sort(ei[ok], 1) == np.sort(d["expert_idx"][ok], 1)).all()


def test_routing_bit_exact_given_logits(case):
    wl, inp, fwd, bwd, logits32, b, dev = case
    s = O.route_spec(oracle_cfg(wl), logits32)
    assert (b.group_idx.cpu().numpy() == s["group_idx"]).all()
    assert (b.expert_idx.cpu().numpy() == s["expert_idx"]).all()
    # the float32 contract also fixes the saved scores
    assert (b.esp.cpu().numpy() == s["ESp"]).all()
    assert (b.gs.cpu().numpy() == s["GS"]).all()
    assert (b.gate_w.cpu().numpy() == s["gate"]).all()
    np.testing.assert_allclose(to_np64(b.gate_w), fwd["gate"], rtol=3e-6)


def test_aux_stats(case):
    wl, inp, fwd, bwd, logits32, b, dev = case
    st = fwd["stats"]
    assert (b.group_count.cpu().numpy() == st["cG"]).all()
    assert (b.cnt_routed.cpu().numpy() == st["cE_route"]).all()
    assert (b.cnt_lit.cpu().numpy() == st["cE_lit"]).all()
    np.testing.assert_allclose(to_np64(b.group_psum), st["sG"], rtol=1e-5)
    np.testing.assert_allclose(to_np64(b.expert_psum), st["sE"], rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(float(b.loss[0]), st["L_G"], rtol=1e-5)
    np.testing.assert_allclose(float(b.loss[1]), st["L_E"], rtol=1e-5)


def test_dispatch_bit_exact(case):
    wl, inp, fwd, bwd, logits32, b, dev = case
    gcfg = gpu_cfg(wl)
    Ne = wl.n_experts
    dp = O.dispatch(fwd["expert_idx"], Ne, gcfg.row_align)
    assert (b.counts.cpu().numpy() == dp["counts"]).all()
    assert (b.offsets.cpu().numpy()[:Ne + 1] == dp["offsets"]).all()
    assert (b.aligned.cpu().numpy()[:Ne + 1] == dp["aligned_offsets"]).all()
    assert (b.row_of.cpu().numpy() == dp["row_of"]).all()
    assert (b.prow_of.cpu().numpy() == dp["prow_of"]).all()
    assert (b.src_of.cpu().numpy() == dp["src_of"]).all()
    rows = int(dp["aligned_offsets"][-1])
    xp = b.x_perm[:rows].cpu()
    want = O.permute_rows(inp["x"].view(torch.int16 if wl.dtype == "bf16" else torch.int32).numpy(),
                          dp["prow_of"], rows)
    got = xp.view(torch.int16 if wl.dtype == "bf16" else torch.int32).numpy()
    assert (got == want).all()                       # bitwise copy, zero padding rows


def test_forward_outputs(case):
    wl, inp, fwd, bwd, logits32, b, dev = case
    tol = tol_for(wl.dtype)
    assert max_rel(to_np64(b.y), fwd["y"]) <= tol
    # per-expert intermediates A, U, H, Y in the permuted layout
    aligned = b.aligned.cpu().numpy()
    for e, c in fwd["per_expert"].items():
        g = e // wl.experts_per_group
        W = wl.group_width[g]
        r0, n = int(aligned[e]), len(c["t"])
        au = to_np64(b.au[r0:r0 + n])
        assert max_rel(au[:, :W], c["A"]) <= tol
        assert max_rel(au[:, W:2 * W], c["U"]) <= tol
        assert max_rel(to_np64(b.h[r0:r0 + n, :W]), c["H"]) <= tol
        assert max_rel(to_np64(b.y_perm[r0:r0 + n]), c["Y"]) <= tol


def test_backward_gradients(case):
    wl, inp, fwd, bwd, logits32, b, dev = case
    tol = tol_for(wl.dtype)
    assert max_rel(to_np64(b.dgate), bwd["dgate"]) <= tol
    assert max_rel(to_np64(b.dlogits), bwd["dlogits"]) <= tol
    assert max_rel(to_np64(b.dx), bwd["dx"]) <= tol
    assert max_rel(to_np64(b.dw_router), bwd["dw_r"]) <= tol
    for g in range(wl.n_groups):
        assert max_rel(to_np64(b.dw13[g]), bwd["dw13"][g]) <= tol, g
        assert max_rel(to_np64(b.dw2[g]), bwd["dw2"][g]) <= tol, g


def test_deterministic_rerun(case):
    wl, inp, fwd, bwd, logits32, b, dev = case
    b2, _ = gpu_layer(wl, inp, logits32=logits32)
    for name in ("group_idx", "expert_idx", "counts", "offsets", "row_of", "prow_of", "src_of",
                 "group_count", "cnt_routed", "cnt_lit"):
        assert torch.equal(getattr(b, name)[:wl.n_experts] if name in ("offsets",) else getattr(b, name),
                           getattr(b2, name)[:wl.n_experts] if name in ("offsets",) else getattr(b2, name)), name
    for name in ("y", "dx", "dw_router", "group_psum", "expert_psum", "loss"):
        a, c = getattr(b, name), getattr(b2, name)
        if name == "loss":
            a, c = a[:2], c[:2]
        assert torch.equal(a, c), name                # same bits run to run
    for g in range(wl.n_groups):
        assert torch.equal(b.dw13[g], b2.dw13[g]) and torch.equal(b.dw2[g], b2.dw2[g])


@pytest.mark.parametrize("switch", ["", "MOHGE_TC_CG=1", "MOHGE_TC_CG=2,MOHGE_TC_WIDE=63",
                                    "MOHGE_FORCE_SIMT=1"])
def test_accumulate_adds_into_weight_gradients(switch):
    """accumulate = 1 adds the weight gradients into dw13 / dw2 (TMA reduce-add in the tensor-core
    forms, read-modify-write in the FFMA kernel); checked in every form of the grouped GEMM."""
    wl = CASES["bf16_small"]
    inp = make_inputs(wl)
    _, _, logits32 = oracle_layer(wl, inp)
    with forced_switches(switch):
        b, dev = gpu_layer(wl, inp, logits32=logits32)
        gcfg = gpu_cfg(wl)
        ref13 = [t.clone() for t in b.dw13]
        ref2 = [t.clone() for t in b.dw2]
        B.layer_backward(gcfg, b, dev["x"], dev["w_router"], dev["w13"], dev["w2"], dev["dy"],
                         aux=True, accumulate=True)
        torch.cuda.synchronize()
    for g in range(wl.n_groups):
        assert max_rel(to_np64(b.dw13[g]), 2 * to_np64(ref13[g])) <= 1e-6
        assert max_rel(to_np64(b.dw2[g]), 2 * to_np64(ref2[g])) <= 1e-6


def test_gate_gradient_from_the_experts_backward_and_from_y_perm(case):
    """The layer's default backward takes the gate gradient out of the SwiGLU-backward epilogue;
    the other route computes <dy, y_perm> in combine_bwd.  Both meet the oracle, and nothing else
    in the backward depends on which one ran."""
    wl, inp, fwd, bwd, logits32, b, dev = case
    tol = tol_for(wl.dtype)
    assert max_rel(to_np64(b.dgate), bwd["dgate"]) <= tol
    fused = {k: getattr(b, k).clone() for k in ("dgate", "dx", "dlogits", "dw_router", "dy_perm", "dau")}
    fused_dw = [t.clone() for t in b.dw13] + [t.clone() for t in b.dw2]
    B.layer_backward(gpu_cfg(wl), b, dev["x"], dev["w_router"], dev["w13"], dev["w2"], dev["dy"],
                     aux=True, fused_dgate=False)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    assert max_rel(to_np64(b.dgate), bwd["dgate"]) <= tol
    assert max_rel(to_np64(b.dgate), to_np64(fused["dgate"])) <= tol
    # same bits either way (compared as integers: columns past a narrow group's width are never
    # written and may hold NaN patterns)
    bits = lambda t: t.view(torch.int16 if t.dtype == torch.bfloat16 else torch.int32)
    for k in ("dy_perm", "dau"):
        assert torch.equal(bits(getattr(b, k)), bits(fused[k])), k
    for t_new, t_old in zip(list(b.dw13) + list(b.dw2), fused_dw):
        assert torch.equal(t_new, t_old)
    # dx, dlogits, dw_router take dgate as an input: equal within the tolerance
    for k in ("dx", "dlogits", "dw_router"):
        assert max_rel(to_np64(getattr(b, k)), to_np64(fused[k])) <= tol, k
