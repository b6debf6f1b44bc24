"""GPU parity at the full benchmark sizes, in the launch configuration the benchmark times.

The inputs are the seeded device-drawn tensors of the benchmark.  Everything integer (group and
expert indices, counts, offsets, permutation, indicator counts) is compared with the oracle in
full for all T tokens.  Floating-point results are compared
  * in full against the oracle where it finishes in tens of seconds (8k- and 16k-token
    workloads), and
  * on the largest workload on what the oracle can evaluate one piece at a time: every output
    row of a random sample of tokens (y, dx, gate and logit gradients, the permuted
    intermediates of their routed copies), every row and both weight gradients of whole sampled
    experts (narrowest and widest group), and the statistics of all tokens.
Bars: bit-exact integers given identical float32 logits; max|a-b|/max|b| <= 2e-2 for BF16, per
tensor and, for the weight gradients, per expert (a cold expert's gradient is much smaller than
a hot one's of the same group).  A second, element-wise figure is printed beside it (run pytest
with -s to see it): the share of elements with |a-b| > tol |b| + tol rms(b).
"""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import WORKLOADS, make_device_inputs

from _util import elementwise_outliers, gpu_cfg, max_rel, oracle_cfg, to_np64

pytestmark = pytest.mark.gpu

TOL = 2e-2
FULL_ORACLE = {"cfg2_bf16": True, "cfg3_bf16_aux": True, "cfg4_bf16_skew": True,
               "cfg5_bf16_large": False, "paper_3b_layer": True, "paper_14b_layer": True,
               "decode_256_large": False, "cfg5_slice": False}
N_SAMPLE_TOKENS = 48


def _run_gpu(wl):
    dev = torch.device("cuda", 0)
    inp = make_device_inputs(wl, dev)
    gcfg = gpu_cfg(wl)
    b = B.LayerBuffers(gcfg, wl.T, device=dev)
    for _ in range(2):          # the second pass runs on warm buffers, as in the benchmark loop
        B.layer_forward(gcfg, b, inp["x"], inp["w_router"], inp["w13"], inp["w2"],
                        logit_bias=inp["logit_bias"], aux=True)
        B.layer_backward(gcfg, b, inp["x"], inp["w_router"], inp["w13"], inp["w2"], inp["dy"],
                         aux=True)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    return gcfg, inp, b


def _close(name, what, got, want, tol=TOL):
    """The bar (max|a-b| / max|b| <= tol) plus the element-wise figure, which is only reported."""
    m = max_rel(got, want)
    print("%s %s: max_rel %.2e, element-wise outliers %.2e" % (name, what, m, elementwise_outliers(got, want, tol)))
    assert m <= tol, (name, what, m)


@pytest.mark.parametrize("name", list(FULL_ORACLE))
def test_full_size_workload(name):
    wl = WORKLOADS[name]
    T, N, Ne, Ke = wl.T, wl.experts_per_group, wl.n_experts, wl.k_experts
    gcfg, inp, b = _run_gpu(wl)
    ocfg = oracle_cfg(wl)
    logits32 = b.logits.cpu().numpy()
    x_cpu, dy_cpu = inp["x"].cpu(), inp["dy"].cpu()
    w_r = to_np64(inp["w_router"])
    bias = None if inp["logit_bias"] is None else to_np64(inp["logit_bias"])

    # ---- integers, all tokens: selection contract, permutation, indicator counts ----
    s = O.route_spec(ocfg, logits32)
    expert_idx = s["expert_idx"]
    assert (b.group_idx.cpu().numpy() == s["group_idx"]).all()
    assert (b.expert_idx.cpu().numpy() == expert_idx).all()
    assert (b.gate_w.cpu().numpy() == s["gate"]).all()
    dp = O.dispatch(expert_idx, Ne, gcfg.row_align)
    assert (b.counts.cpu().numpy() == dp["counts"]).all()
    assert (b.offsets.cpu().numpy()[:Ne + 1] == dp["offsets"]).all()
    assert (b.aligned.cpu().numpy()[:Ne + 1] == dp["aligned_offsets"]).all()
    assert (b.row_of.cpu().numpy() == dp["row_of"]).all()
    assert (b.prow_of.cpu().numpy() == dp["prow_of"]).all()
    assert (b.src_of.cpu().numpy() == dp["src_of"]).all()
    if wl.zipf_beta:
        cnt = dp["counts"]
        ratio = cnt.max() / max(1, cnt.min())      # the skewed workload: counts span about 100x
        print("%s: per-expert token counts %d..%d, ratio %.0f" % (name, cnt.min(), cnt.max(), ratio))
        assert 50 <= ratio <= 200

    # ---- statistics of all tokens (Eq. 7-14) ----
    v = O.route_values(ocfg, logits32.astype(np.float64), s["group_idx"])
    st = O.aux_stats(ocfg, v["GS"], v["ESp"], s["group_idx"], expert_idx, s["ESp"])
    assert (b.group_count.cpu().numpy() == st["cG"]).all()
    assert (b.cnt_routed.cpu().numpy() == st["cE_route"]).all()
    assert (b.cnt_lit.cpu().numpy() == st["cE_lit"]).all()
    np.testing.assert_allclose(to_np64(b.group_psum), st["sG"], rtol=1e-5)
    np.testing.assert_allclose(to_np64(b.expert_psum), st["sE"], rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(float(b.loss[0]), st["L_G"], rtol=1e-5)
    np.testing.assert_allclose(float(b.loss[1]), st["L_E"], rtol=1e-5)
    gate64 = O.gates_from_selection(v["ESpp"], expert_idx)
    aligned = dp["aligned_offsets"]
    prow_of = dp["prow_of"]

    # ---- sampled tokens: every float output that belongs to them ----
    rng = np.random.default_rng(wl.seed + 17)
    tok = np.sort(rng.choice(T, N_SAMPLE_TOKENS, replace=False))
    x_s, dy_s = to_np64(x_cpu[tok]), to_np64(dy_cpu[tok])
    lg = O.router_logits(x_s, w_r, bias)
    assert max_rel(logits32[tok], lg) <= 1e-5
    w13n = [w.cpu().to(torch.float32).numpy() for w in inp["w13"]]
    w2n = [w.cpu().to(torch.float32).numpy() for w in inp["w2"]]
    fs = O.layer_forward(ocfg, x_s, w_r, w13n, w2n, logits=logits32[tok].astype(np.float64), mode="spec")
    cE = st["cE_lit"] if ocfg.fe_mode == 0 else st["cE_route"]
    bs = O.layer_backward(fs, w13n, w2n, dy_s, with_aux=True, aux_counts=(st["cG"], cE, T))
    tok_t = torch.from_numpy(tok).cuda()
    _close(name, "y (sampled tokens)", to_np64(b.y[tok_t]), fs["y"])
    _close(name, "dx (sampled tokens)", to_np64(b.dx[tok_t]), bs["dx"])
    _close(name, "dgate (sampled tokens)", to_np64(b.dgate[tok_t]), bs["dgate"])
    _close(name, "dlogits (sampled tokens)", to_np64(b.dlogits[tok_t]), bs["dlogits"])
    for e, c in fs["per_expert"].items():            # routed copies of the sampled tokens
        W = wl.group_width[e // N]
        rows = torch.from_numpy(prow_of[tok[c["t"]], c["k"]].astype(np.int64)).cuda()
        au = to_np64(b.au[rows])
        assert max_rel(au[:, :W], c["A"]) <= TOL and max_rel(au[:, W:2 * W], c["U"]) <= TOL
        assert max_rel(to_np64(b.h[rows][:, :W]), c["H"]) <= TOL
        assert max_rel(to_np64(b.y_perm[rows]), c["Y"]) <= TOL

    # ---- whole experts: all their rows, both weight gradients ----
    widths = list(wl.group_width)
    for g in sorted({int(np.argmin(widths)), int(np.argmax(widths))}):
        i = int(rng.integers(N))
        if dp["counts"][g * N + i] == 0:                 # tiny batches: take the busiest expert
            i = int(np.argmax(dp["counts"][g * N:(g + 1) * N]))
        e = g * N + i
        W = widths[g]
        t_idx, k_idx = np.nonzero(expert_idx == e)
        n = t_idx.size
        assert n == dp["counts"][e] and n > 0
        xe = to_np64(x_cpu[t_idx])
        w13_e, w2_e = w13n[g][i].astype(np.float64), w2n[g][i].astype(np.float64)
        A, U, H, Y = O.swiglu_ffn(xe, w13_e, w2_e)
        dY = gate64[t_idx, k_idx][:, None] * to_np64(dy_cpu[t_idx])      # derivative of Eq. 15
        eb = O.expert_backward(xe, w13_e, w2_e, A, U, H, dY)
        r0 = int(aligned[e])
        au = to_np64(b.au[r0:r0 + n])
        assert max_rel(au[:, :W], A) <= TOL and max_rel(au[:, W:2 * W], U) <= TOL
        assert max_rel(to_np64(b.h[r0:r0 + n, :W]), H) <= TOL
        assert max_rel(to_np64(b.y_perm[r0:r0 + n]), Y) <= TOL
        assert max_rel(to_np64(b.dy_perm[r0:r0 + n]), dY) <= TOL
        dau = to_np64(b.dau[r0:r0 + n])
        assert max_rel(dau[:, :W], eb["dA"]) <= TOL and max_rel(dau[:, W:2 * W], eb["dU"]) <= TOL
        assert max_rel(to_np64(b.dx_perm[r0:r0 + n]), eb["dx"]) <= TOL
        _close(name, "dw13 of expert %d" % e, to_np64(b.dw13[g][i]), eb["dw13"])
        _close(name, "dw2 of expert %d" % e, to_np64(b.dw2[g][i]), eb["dw2"])
        pad = int(aligned[e + 1]) - r0 - n                               # padding rows stay zero
        if pad:
            assert float(b.x_perm[r0 + n:r0 + n + pad].abs().max()) == 0.0
            assert float(b.dy_perm[r0 + n:r0 + n + pad].abs().max()) == 0.0

    if T <= 1024:
        # few tokens: the forward output of every token (weights converted expert by expert)
        ff = O.layer_forward(ocfg, to_np64(x_cpu), w_r, w13n, w2n, logits=logits32.astype(np.float64),
                             mode="spec")
        assert max_rel(to_np64(b.y), ff["y"]) <= TOL
    # ---- router weight gradient, all tokens: dW_r = dlogits^T x in fp64 from the GPU's own
    # dlogits (checked against the oracle on the sampled tokens above and, where the full oracle
    # runs, in full below); this pins the split-K sum over the tokens at every batch size ----
    dl = to_np64(b.dlogits)
    dw_r = np.zeros((wl.n_logits, wl.d_model))
    for t0 in range(0, T, 8192):
        dw_r += dl[t0:t0 + 8192].T @ to_np64(x_cpu[t0:t0 + 8192])
    _close(name, "dw_router (from the GPU's dlogits)", to_np64(b.dw_router), dw_r)
    if not FULL_ORACLE[name]:
        return
    # ---- every element against the full oracle ----
    w13d = [w.astype(np.float64) for w in w13n]
    w2d = [w.astype(np.float64) for w in w2n]
    fwd = O.layer_forward(ocfg, to_np64(x_cpu), w_r, w13d, w2d, logits=logits32.astype(np.float64),
                          mode="spec")
    bwd = O.layer_backward(fwd, w13d, w2d, to_np64(dy_cpu), with_aux=True)
    _close(name, "y", to_np64(b.y), fwd["y"])
    _close(name, "dx", to_np64(b.dx), bwd["dx"])
    _close(name, "dgate", to_np64(b.dgate), bwd["dgate"])
    _close(name, "dlogits", to_np64(b.dlogits), bwd["dlogits"])
    _close(name, "dw_router", to_np64(b.dw_router), bwd["dw_r"])
    for g in range(wl.n_groups):
        dw13, dw2 = to_np64(b.dw13[g]), to_np64(b.dw2[g])
        assert max_rel(dw13, bwd["dw13"][g]) <= TOL, g
        assert max_rel(dw2, bwd["dw2"][g]) <= TOL, g
        for i in range(N):                           # per expert: cold experts have small gradients
            assert max_rel(dw13[i], bwd["dw13"][g][i]) <= TOL, (g, i)
            assert max_rel(dw2[i], bwd["dw2"][g][i]) <= TOL, (g, i)
