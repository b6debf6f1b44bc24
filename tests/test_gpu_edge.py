"""GPU edge cases: degenerate routing (all ties, every token to one expert, empty experts),
single token, empty batch, K_g sweep, maximum slot count."""
import numpy as np
import pytest
import torch

import oracle as O
from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import Workload, make_inputs

from _util import forced_switches, gpu_cfg, gpu_layer, max_rel, oracle_cfg, oracle_layer, to_np64, tol_for

pytestmark = pytest.mark.gpu


def _compare(wl, inp, logits32):
    fwd, bwd, _ = oracle_layer(wl, inp, logits32=logits32)
    b, dev = gpu_layer(wl, inp, logits32=logits32)
    tol = tol_for(wl.dtype)
    assert (b.expert_idx.cpu().numpy() == fwd["expert_idx"]).all()
    assert (b.group_idx.cpu().numpy() == fwd["group_idx"]).all()
    dp = O.dispatch(fwd["expert_idx"], wl.n_experts, gpu_cfg(wl).row_align)
    assert (b.counts.cpu().numpy() == dp["counts"]).all()
    assert (b.prow_of.cpu().numpy() == dp["prow_of"]).all()
    assert (b.src_of.cpu().numpy() == dp["src_of"]).all()
    assert max_rel(to_np64(b.y), fwd["y"]) <= tol
    assert max_rel(to_np64(b.dx), bwd["dx"]) <= tol
    assert max_rel(to_np64(b.dw_router), bwd["dw_r"]) <= tol
    for g in range(wl.n_groups):
        assert max_rel(to_np64(b.dw13[g]), bwd["dw13"][g]) <= tol
        assert max_rel(to_np64(b.dw2[g]), bwd["dw2"][g]) <= tol
    return fwd, b


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_all_logits_equal_ties_go_to_lowest_index(dtype):
    wl = Workload("ties", dtype, 300, 64, 3, 4, (64, 32, 48), 2, 6, seed=7)
    inp = make_inputs(wl)
    logits = np.zeros((wl.T, wl.n_logits), np.float32)
    fwd, b = _compare(wl, inp, logits)
    assert (fwd["expert_idx"] == np.arange(6)).all()          # experts 0..5, half of them empty after
    assert (b.counts.cpu().numpy()[6:] == 0).all()
    for g in (2,):                                            # empty experts: exactly zero gradients
        assert float(b.dw13[g].abs().max()) == 0.0 and float(b.dw2[g].abs().max()) == 0.0


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_every_token_to_one_expert_set(dtype):
    wl = Workload("funnel", dtype, 700, 64, 2, 8, (96, 40), 1, 2, seed=8)
    inp = make_inputs(wl)
    logits = np.zeros((wl.T, wl.n_logits), np.float32)
    logits[:, 1] = 3.0                    # group 1 always wins
    logits[:, 2 + 8 + 5] = 4.0            # its expert 5 first, expert 2 second
    logits[:, 2 + 8 + 2] = 2.0
    fwd, b = _compare(wl, inp, logits)
    cnt = b.counts.cpu().numpy()
    assert cnt[13] == wl.T and cnt[10] == wl.T and cnt.sum() == 2 * wl.T


@pytest.mark.parametrize("dtype,T", [("f32", 1), ("bf16", 1), ("bf16", 129), ("f32", 257)])
def test_tiny_batches(dtype, T):
    wl = Workload("tiny", dtype, T, 64, 2, 4, (64, 32), 1, 2, seed=9)
    inp = make_inputs(wl)
    _, _, logits32 = oracle_layer(wl, inp)
    _compare(wl, inp, logits32)


@pytest.mark.parametrize("K_g", [1, 2, 3, 4])
def test_group_budget_sweep(K_g):
    wl = Workload("kg", "f32", 200, 32, 4, 4, (32, 24, 16, 8), K_g, min(6, 4 * K_g), seed=10)
    inp = make_inputs(wl)
    _, _, logits32 = oracle_layer(wl, inp)
    _compare(wl, inp, logits32)


def test_maximum_router_width():
    # N_g = 8 groups of N = 32 experts: 256 expert slots, 8 per lane; K_e = 32 fills every lane
    wl = Workload("max", "f32", 150, 32, 8, 32, (8,) * 8, 3, 32, seed=11)
    inp = make_inputs(wl)
    _, _, logits32 = oracle_layer(wl, inp)
    _compare(wl, inp, logits32)


def test_empty_batch_launches_nothing_and_zeroes_statistics():
    wl = Workload("empty", "f32", 0, 32, 2, 4, (32, 16), 1, 2)
    gcfg = gpu_cfg(wl)
    b = B.LayerBuffers(gcfg, 0)
    x = torch.zeros(1, 32, device="cuda")
    wr = torch.zeros(wl.n_logits, 32, device="cuda")
    w13 = [torch.zeros(4, 2 * w, 32, device="cuda") for w in wl.group_width]
    w2 = [torch.zeros(4, 32, w, device="cuda") for w in wl.group_width]
    B.layer_forward(gcfg, b, x, wr, w13, w2)
    B.layer_backward(gcfg, b, x, wr, w13, w2, x)
    torch.cuda.synchronize()
    assert int(b.counts.sum()) == 0 and int(b.aligned[wl.n_experts]) == 0
    assert float(b.dw_router.abs().max()) == 0.0
    assert all(float(t.abs().max()) == 0.0 for t in b.dw13 + b.dw2)
    assert B.mohge_get_device_status(b.ws) == 0


def test_out_of_range_expert_index_sets_the_status_word_without_faulting():
    wl = Workload("badidx", "f32", 64, 32, 2, 4, (32, 16), 1, 2)
    gcfg = gpu_cfg(wl)
    b = B.LayerBuffers(gcfg, 64)
    x = torch.zeros(64, 32, device="cuda")
    idx = torch.zeros(64, 2, dtype=torch.int32, device="cuda")
    idx[:, 1] = 1
    idx[5, 1] = 99                                    # not an expert: skipped and reported
    B.mohge_dispatch(gcfg, 64, x, idx, b.counts, b.offsets, b.aligned, b.row_of, b.prow_of,
                     b.src_of, b.x_perm, b.ws)
    torch.cuda.synchronize()
    rc, word = B.mohge_get_device_status_rc(b.ws)
    assert word >> 24 == 2 and rc == B.MOHGE_ERR_DEVICE_CHECK      # decoded from the word
    assert b"index check" in B.lib().mohge_last_error()
    assert int(b.counts.sum()) == 127


def test_nan_logits_rank_below_every_number_and_are_reported():
    """NaN router logits are invalid input: they lose against every number (ties among them to
    the lowest index), the indices still equal the oracle's under that reading bit for bit, and
    the status word says so."""
    wl = Workload("nan_logits", "f32", 300, 32, 3, 4, (32, 24, 16), 2, 5, seed=4)
    gcfg, ocfg = gpu_cfg(wl), oracle_cfg(wl)
    rng = np.random.default_rng(12)
    lg = rng.normal(size=(wl.T, wl.n_logits)).astype(np.float32)
    nan_at = rng.random(lg.shape) < 0.15
    nan_at[0] = True
    nan_at[1, :3] = True
    nan_at[2, 3:7] = True
    lg[nan_at] = np.nan
    s = O.route_spec(ocfg, lg)
    assert s["nan_logits"] == int(nan_at.sum())
    b = B.LayerBuffers(gcfg, wl.T)
    B.mohge_route(gcfg, wl.T, None, None, None, torch.from_numpy(lg).cuda(), None, b.group_idx,
                  b.expert_idx, b.gate_w, b.gs, b.esp, b.ws)
    torch.cuda.synchronize()
    assert (b.group_idx.cpu().numpy() == s["group_idx"]).all()
    assert (b.expert_idx.cpu().numpy() == s["expert_idx"]).all()
    ok = ~nan_at[:, :3].any(axis=1)                      # tokens whose group logits are numbers
    assert (b.gate_w.cpu().numpy()[ok] == s["gate"][ok]).all()
    rc, word = B.mohge_get_device_status_rc(b.ws)
    assert word == 3 << 24 and rc == B.MOHGE_ERR_DEVICE_CHECK
    assert b"NaN" in B.lib().mohge_last_error()
    # a batch without NaN leaves the word alone
    B.mohge_workspace_init(gcfg, wl.T, b.ws)
    B.mohge_route(gcfg, wl.T, None, None, None, torch.from_numpy(np.nan_to_num(lg)).cuda(), None,
                  b.group_idx, b.expert_idx, b.gate_w, b.gs, b.esp, b.ws)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status_rc(b.ws) == (0, 0)


def test_tensor_maps_are_encoded_once_per_launch_site():
    """A layer stepped on the same buffers encodes its TMA tensor maps on the first step only."""
    wl = Workload("map_cache", "bf16", 700, 256, 3, 4, (352, 176, 88), 2, 4, seed=3)
    inp = make_inputs(wl)
    gcfg = gpu_cfg(wl)
    dev = {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in inp.items() if k not in ("w13", "w2")}
    w13, w2 = [w.cuda() for w in inp["w13"]], [w.cuda() for w in inp["w2"]]
    b = B.LayerBuffers(gcfg, wl.T)

    def step():
        B.layer_forward(gcfg, b, dev["x"], dev["w_router"], w13, w2, aux=True)
        B.layer_backward(gcfg, b, dev["x"], dev["w_router"], w13, w2, dev["dy"], aux=True)

    step()
    h0, m0 = B.mohge_map_cache_stats()
    step()
    step()
    torch.cuda.synchronize()
    h1, m1 = B.mohge_map_cache_stats()
    assert m1 == m0                                     # no new encodes
    assert h1 - h0 == 2 * 9                             # nine tensor-core GEMM launches per step
    y = b.y.clone()
    step()
    torch.cuda.synchronize()
    assert torch.equal(y, b.y) and B.mohge_get_device_status(b.ws) == 0


@pytest.mark.skipif(not torch.cuda.is_available() or torch.cuda.device_count() < 2,
                    reason="needs two visible GPUs")
def test_layer_on_a_second_device_of_the_same_process():
    """Kernel attributes, SM count and cached tensor maps are kept per device ordinal: a process
    that has already used device 0 runs the same layer on device 1 and gets the same bits."""
    wl = Workload("second_device", "bf16", 600, 256, 3, 4, (352, 176, 88), 2, 4, seed=6)
    inp = make_inputs(wl)
    gcfg = gpu_cfg(wl)
    outs = []
    for ordinal in (0, 1):
        with torch.cuda.device(ordinal):
            d = torch.device("cuda", ordinal)
            x, w_r, dy = inp["x"].to(d), inp["w_router"].to(d), inp["dy"].to(d)
            w13, w2 = [w.to(d) for w in inp["w13"]], [w.to(d) for w in inp["w2"]]
            b = B.LayerBuffers(gcfg, wl.T, device=d)
            B.layer_forward(gcfg, b, x, w_r, w13, w2, aux=True)
            B.layer_backward(gcfg, b, x, w_r, w13, w2, dy, aux=True)
            torch.cuda.synchronize()
            assert B.mohge_get_device_status(b.ws) == 0
            outs.append((b.y.cpu(), b.dx.cpu(), b.dw13[0].cpu()))
    for a, c in zip(*outs):
        assert torch.equal(a, c)


@pytest.mark.parametrize("switch", ["MOHGE_TC_CG=2,MOHGE_TC_WIDE=63", "MOHGE_TC_CG=2,MOHGE_TC_WIDE=0",
                                    "MOHGE_TC_CG=1", "MOHGE_PDL=0", "MOHGE_FORCE_SIMT=1"])
def test_every_form_of_the_grouped_gemm_on_small_ragged_cases(switch):
    """The double-width form is chosen by default only for long contractions (the large
    workload) and single CTAs only for batches with few rows per expert, and the GEMM kernels are
    launched as programmatic dependents of their predecessors unless switched off; here each form is forced
    on small ragged shapes, so that every kernel form meets odd widths, ragged tails, empty experts
    and both a few and a few hundred rows per expert."""
    with forced_switches(switch):
        for wl in (Workload("forms_a", "bf16", 1000, 256, 3, 4, (352, 176, 88), 2, 4, seed=1),
                   Workload("forms_few", "bf16", 90, 256, 3, 4, (352, 176, 88), 2, 4, seed=2),
                   Workload("forms_b", "bf16", 1500, 256, 4, 8, (256, 192, 128, 64), 2, 6,
                            zipf_beta=3.0, seed=5)):
            inp = make_inputs(wl)
            _, _, logits32 = oracle_layer(wl, inp)
            _compare(wl, inp, logits32)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_single_expert_layer_is_a_plain_ffn(dtype):
    """N_g = N = K_g = K_e = 1: the gate is 1 for every token, so y is the expert's FFN of x and
    the router receives no gradient beyond float32 cancellation noise (the exact value is of the
    order of eps, far below anything a relative bar could be applied to)."""
    wl = Workload("one_expert", dtype, 257, 64, 1, 1, (344,), 1, 1, seed=9)
    inp = make_inputs(wl)
    fwd, bwd, logits32 = oracle_layer(wl, inp)
    b, dev = gpu_layer(wl, inp, logits32=logits32)
    tol = tol_for(dtype)
    assert (b.gate_w.cpu().numpy() == 1.0).all() and (b.expert_idx.cpu().numpy() == 0).all()
    A, U, H, Y = O.swiglu_ffn(to_np64(inp["x"]), to_np64(inp["w13"][0][0]), to_np64(inp["w2"][0][0]))
    assert max_rel(to_np64(b.y), Y) <= tol and max_rel(fwd["y"], Y) <= 1e-12
    assert max_rel(to_np64(b.dx), bwd["dx"]) <= tol
    assert max_rel(to_np64(b.dw13[0]), bwd["dw13"][0]) <= tol
    assert max_rel(to_np64(b.dw2[0]), bwd["dw2"][0]) <= tol
    assert max_rel(to_np64(b.dgate), bwd["dgate"]) <= tol
    scale = float(np.abs(bwd["dgate"]).max())
    assert np.abs(bwd["dlogits"]).max() <= 1e-12 * scale
    assert float(b.dlogits.abs().max()) <= 1e-6 * scale
    assert float(b.dw_router.abs().max()) <= 1e-6 * scale * wl.T


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_gate_that_is_exactly_zero_still_gets_its_gradient(dtype):
    """One of the two selected experts has a score that underflows to 0 in the float32 contract,
    so its gate is exactly 0 and its row of dy_perm is zero; its gate gradient <dy, Y> is not."""
    wl = Workload("zero_gate", dtype, 200, 64, 1, 2, (96,), 1, 2, seed=11)
    inp = make_inputs(wl)
    logits = np.zeros((wl.T, wl.n_logits), np.float32)
    logits[:, 2] = -200.0                      # second expert: exp_s(-200) = 0
    fwd, bwd, _ = oracle_layer(wl, inp, logits32=logits)
    b, dev = gpu_layer(wl, inp, logits32=logits)
    g = b.gate_w.cpu().numpy()
    assert (g[:, 0] == 1.0).all() and (g[:, 1] == 0.0).all()
    assert (b.expert_idx.cpu().numpy() == fwd["expert_idx"]).all()
    assert np.abs(bwd["dgate"][:, 1]).max() > 0
    assert max_rel(to_np64(b.dgate), bwd["dgate"]) <= tol_for(dtype)
    assert max_rel(to_np64(b.y), fwd["y"]) <= tol_for(dtype)


@pytest.mark.parametrize("T", [148 * 128 + 1, 20000, 148 * 192, 33333])
def test_router_logits_with_more_row_tiles_than_sms(T):
    """With more 128-row tiles than SMs the logits GEMM gives every CTA one contiguous range of
    rows, the last tile of a range being 64 rows high: every row must still be computed once,
    whatever the remainder, and the selection from those logits must be the contract's."""
    wl = Workload("balanced_logits", "bf16", T, 192, 3, 8, (64, 48, 32), 2, 4, seed=13)
    inp = make_inputs(wl, weights=False)
    gcfg, ocfg = gpu_cfg(wl), oracle_cfg(wl)
    b = B.LayerBuffers(gcfg, T)
    b.logits.fill_(float("nan"))
    B.mohge_route(gcfg, T, inp["x"].cuda(), inp["w_router"].cuda(), None, None, b.logits, b.group_idx,
                  b.expert_idx, b.gate_w, b.gs, b.esp, b.ws)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    ref = O.router_logits(to_np64(inp["x"]), to_np64(inp["w_router"]), None)
    got = b.logits.cpu().numpy()
    assert np.isfinite(got).all()
    assert max_rel(got, ref) <= 1e-5
    s = O.route_spec(ocfg, got)
    assert (b.group_idx.cpu().numpy() == s["group_idx"]).all()
    assert (b.expert_idx.cpu().numpy() == s["expert_idx"]).all()


@pytest.mark.parametrize("shape", [(3, 4, 2, 5), (4, 32, 2, 8), (8, 32, 3, 20), (2, 7, 2, 14), (1, 1, 1, 1), (5, 3, 5, 15)])
def test_selection_contract_on_ties_nan_and_underflow(shape):
    """Indices, gates and saved scores equal the oracle's float32 contract bit for bit on rows
    full of exact ties, rows where everything ties, NaN group logits, groups of NaN expert logits
    and scores that underflow to zero (rows whose keys all underflow have 0/0 gates on both sides)."""
    Ng, N, Kg, Ke = shape
    wl = Workload("contract_edges", "f32", 1000, 32, Ng, N, tuple([32] * Ng), Kg, Ke, seed=21)
    gcfg, ocfg = gpu_cfg(wl), oracle_cfg(wl)
    rng = np.random.default_rng(7)
    lg = rng.normal(size=(wl.T, wl.n_logits)).astype(np.float32)
    lg[:100] = np.round(lg[:100] * 2) / 2                  # many exact ties
    lg[100:110] = 0.0                                      # everything ties
    lg[110:120, 0] = np.nan                                # NaN group logit
    lg[120:130, Ng:] = np.nan                              # all expert logits NaN
    lg[130:140] = -200.0 * (rng.random((10, wl.n_logits)) < 0.5)   # underflowing scores
    s = O.route_spec(ocfg, lg)
    b = B.LayerBuffers(gcfg, wl.T)
    B.mohge_route(gcfg, wl.T, None, None, None, torch.from_numpy(lg).cuda(), None, b.group_idx,
                  b.expert_idx, b.gate_w, b.gs, b.esp, b.ws)
    torch.cuda.synchronize()
    assert (b.group_idx.cpu().numpy() == s["group_idx"]).all()
    assert (b.expert_idx.cpu().numpy() == s["expert_idx"]).all()
    assert np.array_equal(b.gate_w.cpu().numpy(), s["gate"], equal_nan=True)
    assert np.array_equal(b.esp.cpu().numpy(), s["ESp"], equal_nan=True)
    assert np.array_equal(b.gs.cpu().numpy(), s["GS"], equal_nan=True)
