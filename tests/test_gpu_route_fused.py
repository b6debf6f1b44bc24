"""mohge_route with the selection done in the epilogue of the logits GEMM (one thread per token on
the accumulator rows) against the two-kernel route and against the oracle's float32 contract."""
import numpy as np
import pytest
import torch

from oracle import mohge_oracle as O
from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import Workload, make_inputs

from _util import forced_switches, gpu_cfg, max_rel, oracle_cfg, to_np64

pytestmark = pytest.mark.gpu

OUT = ("logits", "group_idx", "expert_idx", "gate_w", "gs", "esp")


def _route(gcfg, T, x, w, bias, fill=None):
    b = B.LayerBuffers(gcfg, T)
    if fill is not None:
        b.logits.fill_(fill)
        b.esp.fill_(fill)
    n0 = B.mohge_launch_count()
    B.mohge_route(gcfg, T, x, w, bias, None, b.logits, b.group_idx, b.expert_idx, b.gate_w, b.gs, b.esp, b.ws)
    torch.cuda.synchronize()
    return b, B.mohge_launch_count() - n0


def _both(gcfg, T, x, w, bias):
    with forced_switches("MOHGE_ROUTE_FUSED=0"):
        two, n_two = _route(gcfg, T, x, w, bias)
    one, n_one = _route(gcfg, T, x, w, bias, fill=float("nan"))
    return one, n_one, two, n_two


# (Ng, N, Kg, Ke)
SHAPES = [(4, 32, 2, 8), (4, 16, 2, 6), (8, 8, 3, 8), (8, 16, 2, 8), (4, 4, 2, 8), (3, 8, 2, 4), (2, 4, 1, 2),
          (4, 32, 4, 8), (1, 32, 1, 8), (2, 8, 2, 1)]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("T", [5000, 148 * 128 + 77])
@pytest.mark.parametrize("with_bias", [False, True])
def test_fused_route_is_the_two_kernel_route_bit_for_bit(shape, T, with_bias):
    Ng, N, Kg, Ke = shape
    wl = Workload("route_fused", "bf16", T, 320, Ng, N, tuple([64] * Ng), Kg, Ke, seed=31 + Ng + N)
    inp = make_inputs(wl, weights=False)
    gcfg, ocfg = gpu_cfg(wl), oracle_cfg(wl)
    x, w = inp["x"].cuda(), (inp["w_router"] * 20).cuda()        # logits of order one
    bias = None
    if with_bias:
        g = torch.Generator().manual_seed(5)
        bias = torch.randn(wl.n_logits, generator=g).cuda()
    one, n_one, two, n_two = _both(gcfg, T, x, w, bias)
    assert n_one == n_two - 1                                    # the selection kernel is gone
    assert B.mohge_get_device_status(one.ws) == 0
    for name in OUT:
        a, c = getattr(one, name).cpu().numpy(), getattr(two, name).cpu().numpy()
        assert np.array_equal(a, c), name
    got = one.logits.cpu().numpy()
    ref = O.router_logits(to_np64(x.cpu()), to_np64(w.cpu()), None if bias is None else to_np64(bias.cpu()))
    assert max_rel(got, ref) <= 1e-5
    s = O.route_spec(ocfg, got)
    assert (one.group_idx.cpu().numpy() == s["group_idx"]).all()
    assert (one.expert_idx.cpu().numpy() == s["expert_idx"]).all()
    assert np.array_equal(one.gate_w.cpu().numpy(), s["gate"])
    assert np.array_equal(one.esp.cpu().numpy(), s["ESp"])
    assert np.array_equal(one.gs.cpu().numpy(), s["GS"])


@pytest.mark.parametrize("shape", [(4, 32, 2, 8), (8, 16, 3, 8), (3, 8, 2, 5), (4, 4, 4, 8)])
def test_fused_route_on_ties_and_underflow(shape):
    """Rows of x that are unit vectors make row t of the logits a column of the router weight, so
    the logits can be set exactly: rows full of ties, rows where everything ties, scores that
    underflow to zero.  The fused selection must give the contract's indices, gates and scores."""
    Ng, N, Kg, Ke = shape
    d, T = 256, 6000
    wl = Workload("route_fused_edges", "bf16", T, d, Ng, N, tuple([64] * Ng), Kg, Ke, seed=3)
    gcfg, ocfg = gpu_cfg(wl), oracle_cfg(wl)
    rng = np.random.default_rng(11)
    NL = wl.n_logits
    table = rng.normal(size=(d, NL)).astype(np.float32)
    table[:100] = np.round(table[:100] * 2) / 2                    # many exact ties
    table[100:110] = 0.0                                           # everything ties
    table[110:120] = -200.0 * (rng.random((10, NL)) < 0.5)         # underflowing scores
    table[120:130] = np.where(rng.random((10, NL)) < 0.5, 0.0, -0.0)
    w = torch.from_numpy(table.T.copy()).to(torch.bfloat16)        # [NL, d]
    x = torch.zeros(T, d, dtype=torch.bfloat16)
    x[torch.arange(T), torch.arange(T) % d] = 1.0
    one, n_one, two, n_two = _both(gcfg, T, x.cuda(), w.cuda(), None)
    assert n_one == n_two - 1
    got = one.logits.cpu().numpy()
    assert np.array_equal(got, w.float().numpy().T[np.arange(T) % d])
    for name in OUT:
        a, c = getattr(one, name).cpu().numpy(), getattr(two, name).cpu().numpy()
        assert np.array_equal(a, c, equal_nan=True), name
    s = O.route_spec(ocfg, got)
    assert (one.group_idx.cpu().numpy() == s["group_idx"]).all()
    assert (one.expert_idx.cpu().numpy() == s["expert_idx"]).all()
    assert np.array_equal(one.gate_w.cpu().numpy(), s["gate"], equal_nan=True)
    assert np.array_equal(one.esp.cpu().numpy(), s["ESp"], equal_nan=True)
    assert np.array_equal(one.gs.cpu().numpy(), s["GS"], equal_nan=True)


@pytest.mark.parametrize("where", ["x_row", "bias_group", "bias_expert"])
def test_fused_route_reads_nan_logits_as_lowest_and_reports_them(where):
    wl = Workload("route_fused_nan", "bf16", 6000, 128, 4, 16, (64, 64, 64, 64), 2, 6, seed=9)
    inp = make_inputs(wl, weights=False)
    gcfg, ocfg = gpu_cfg(wl), oracle_cfg(wl)
    x, w = inp["x"].clone(), inp["w_router"] * 20
    bias = torch.zeros(wl.n_logits)
    if where == "x_row":
        x[17, 5] = float("nan")
        x[5999, 0] = float("nan")
    elif where == "bias_group":
        bias[1] = float("nan")
    else:
        bias[4 + 16 * 2 + 3] = float("nan")
    one, n_one, two, n_two = _both(gcfg, wl.T, x.cuda(), w.cuda(), bias.cuda())
    assert n_one == n_two - 1
    assert B.mohge_get_device_status(one.ws) == (3 << 24)
    assert B.mohge_get_device_status_rc(one.ws)[0] == B.MOHGE_ERR_DEVICE_CHECK
    got = one.logits.cpu().numpy()
    assert np.isnan(got).any()
    s = O.route_spec(ocfg, got)
    assert s["nan_logits"] > 0
    for name in OUT:
        a, c = getattr(one, name).cpu().numpy(), getattr(two, name).cpu().numpy()
        assert np.array_equal(a, c, equal_nan=True), name
    assert (one.group_idx.cpu().numpy() == s["group_idx"]).all()
    assert (one.expert_idx.cpu().numpy() == s["expert_idx"]).all()
    assert np.array_equal(one.gate_w.cpu().numpy(), s["gate"], equal_nan=True)
    assert np.array_equal(one.esp.cpu().numpy(), s["ESp"], equal_nan=True)
