"""Pins for the oracle's experts, combine and backward: dense library special
cases, autograd of an independently written dense forward, finite differences."""
import numpy as np
import pytest
import torch

import oracle as O


def _rand_layer(cfg, T, seed, scale=0.3):
    rng = np.random.default_rng(seed)
    d, N = cfg.d_model, cfg.experts_per_group
    x = rng.normal(size=(T, d))
    w_r = rng.normal(size=(cfg.n_groups + cfg.n_experts, d)) * scale
    w13 = [rng.normal(size=(N, 2 * W, d)) * scale for W in cfg.group_width]
    w2 = [rng.normal(size=(N, d, W)) * scale for W in cfg.group_width]
    dy = rng.normal(size=(T, d))
    return x, w_r, w13, w2, dy


def test_single_expert_is_a_dense_swiglu_ffn():
    cfg = O.OracleConfig(d_model=12, n_groups=1, experts_per_group=1, k_groups=1, k_experts=1,
                         group_width=[20])
    x, w_r, w13, w2, dy = _rand_layer(cfg, 9, 0)
    f = O.layer_forward(cfg, x, w_r, w13, w2)
    np.testing.assert_allclose(f["gate"], 1.0)
    tx = torch.tensor(x)
    wg, wu, wd = torch.tensor(w13[0][0][:20]), torch.tensor(w13[0][0][20:]), torch.tensor(w2[0][0])
    ref = (torch.nn.functional.silu(tx @ wg.T) * (tx @ wu.T)) @ wd.T
    np.testing.assert_allclose(f["y"], ref.numpy(), rtol=1e-12, atol=1e-13)


def test_expert_backward_matches_autograd_of_a_dense_swiglu_ffn():
    rng = np.random.default_rng(3)
    n, d, W = 7, 10, 6
    x, w13, w2, dY = (rng.normal(size=s) for s in ((n, d), (2 * W, d), (d, W), (n, d)))
    A, U, H, Y = O.swiglu_ffn(x, w13, w2)
    got = O.expert_backward(x, w13, w2, A, U, H, dY)
    tx, t13, t2 = (torch.tensor(a, requires_grad=True) for a in (x, w13, w2))
    ty = (torch.nn.functional.silu(tx @ t13[:W].T) * (tx @ t13[W:].T)) @ t2.T
    (ty * torch.tensor(dY)).sum().backward()
    np.testing.assert_allclose(Y, ty.detach().numpy(), rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(got["dx"], tx.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(got["dw13"], t13.grad.numpy(), rtol=1e-10, atol=1e-12)
    np.testing.assert_allclose(got["dw2"], t2.grad.numpy(), rtol=1e-10, atol=1e-12)


def _torch_dense_forward(cfg, x, w_r, w13, w2, G):
    """Independent forward: every expert is evaluated on every token and mixed
    with a dense [T, N_e] gate matrix built with torch.topk / torch.softmax."""
    N_g, N, N_e = cfg.n_groups, cfg.experts_per_group, cfg.n_experts
    T = x.shape[0]
    logits = x @ w_r.T
    GS = torch.sigmoid(logits[:, :N_g])
    gmask = torch.zeros(T, N_g, dtype=torch.bool)
    gmask.scatter_(1, torch.topk(GS, cfg.k_groups, dim=1).indices, True)
    ESp = torch.softmax(logits[:, N_g:].reshape(T, N_g, N), dim=2) * gmask[:, :, None]
    ESpp = (ESp * GS[:, :, None]).reshape(T, N_e)
    top = torch.topk(ESpp, cfg.k_experts, dim=1)
    emask = torch.zeros(T, N_e, dtype=torch.bool)
    emask.scatter_(1, top.indices, True)
    ES3 = ESpp * emask
    ES = ES3 / ES3.sum(1, keepdim=True)
    y = torch.zeros_like(x)
    for e in range(N_e):
        g, i = divmod(e, N)
        W = cfg.group_width[g]
        h = torch.nn.functional.silu(x @ w13[g][i][:W].T) * (x @ w13[g][i][W:].T)
        y = y + ES[:, e:e + 1] * (h @ w2[g][i].T)
    # auxiliary losses; the indicator frequencies are constants
    Wd = torch.tensor(cfg.group_width, dtype=torch.float64)
    fG = (N_g / cfg.k_groups) * gmask.sum(0).double() / T
    pG = (GS / GS.sum(1, keepdim=True)).mean(0)
    L_G = cfg.alpha_g * torch.sum(Wd / Wd.max() * fG * pG)
    ESp_flat = ESp.reshape(T, N_e)
    if cfg.fe_mode == 0:
        lit = torch.zeros(T, N_e, dtype=torch.bool)
        lit.scatter_(1, torch.topk(ESp_flat.detach(), cfg.k_experts, dim=1).indices, True)
        cE = lit.sum(0).double()
    else:
        cE = emask.sum(0).double()
    fE = (N / cfg.k_experts) * cE / T
    SE = ESp / (ESp.sum(2, keepdim=True) + cfg.eps)
    pE = SE.reshape(T, N_e).mean(0)
    L_E = cfg.alpha_e * torch.sum(fE * pE)
    return y, torch.sum(y * G) + L_G + L_E, L_G, L_E


@pytest.mark.parametrize("N_g,N,K_g,K_e,widths,fe_mode", [
    (2, 4, 1, 2, [24, 12], 0), (3, 3, 2, 4, [8, 16, 24], 1), (2, 2, 2, 4, [10, 6], 0)])
def test_forward_and_backward_match_torch_autograd(N_g, N, K_g, K_e, widths, fe_mode):
    # large alphas so that the auxiliary terms are visible in the gradients
    cfg = O.OracleConfig(d_model=10, n_groups=N_g, experts_per_group=N, k_groups=K_g,
                         k_experts=K_e, group_width=widths, alpha_g=0.7, alpha_e=0.9,
                         fe_mode=fe_mode)
    T = 40
    x, w_r, w13, w2, dy = _rand_layer(cfg, T, 21)
    f = O.layer_forward(cfg, x, w_r, w13, w2)
    b = O.layer_backward(f, w13, w2, dy, with_aux=True)
    tx = torch.tensor(x, requires_grad=True)
    twr = torch.tensor(w_r, requires_grad=True)
    tw13 = [torch.tensor(w, requires_grad=True) for w in w13]
    tw2 = [torch.tensor(w, requires_grad=True) for w in w2]
    y, loss, L_G, L_E = _torch_dense_forward(cfg, tx, twr, tw13, tw2, torch.tensor(dy))
    loss.backward()
    np.testing.assert_allclose(f["y"], y.detach().numpy(), rtol=1e-11, atol=1e-12)
    np.testing.assert_allclose(f["stats"]["L_G"], float(L_G.detach()), rtol=1e-12)
    np.testing.assert_allclose(f["stats"]["L_E"], float(L_E.detach()), rtol=1e-12)
    np.testing.assert_allclose(O.layer_loss(f, dy), float(loss.detach()), rtol=1e-12)
    tol = dict(rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(b["dx"], tx.grad.numpy(), **tol)
    np.testing.assert_allclose(b["dw_r"], twr.grad.numpy(), **tol)
    for g in range(N_g):
        np.testing.assert_allclose(b["dw13"][g], tw13[g].grad.numpy(), **tol)
        np.testing.assert_allclose(b["dw2"][g], tw2[g].grad.numpy(), **tol)
    # without the auxiliary terms: gradient of <y, dy> alone
    b0 = O.layer_backward(f, w13, w2, dy, with_aux=False)
    for t_ in (tx, twr):
        t_.grad = None
    y2, _, _, _ = _torch_dense_forward(cfg, tx, twr, tw13, tw2, torch.tensor(dy))
    torch.sum(y2 * torch.tensor(dy)).backward()
    np.testing.assert_allclose(b0["dx"], tx.grad.numpy(), **tol)
    np.testing.assert_allclose(b0["dw_r"], twr.grad.numpy(), **tol)


def test_backward_matches_central_finite_differences():
    cfg = O.OracleConfig(d_model=6, n_groups=2, experts_per_group=3, k_groups=1, k_experts=2,
                         group_width=[8, 4], alpha_g=0.5, alpha_e=0.5)
    T = 12
    x, w_r, w13, w2, dy = _rand_layer(cfg, T, 5)
    f = O.layer_forward(cfg, x, w_r, w13, w2)
    # routing margins must be wide enough that a 1e-6 perturbation flips nothing
    GS = np.sort(f["GS"], 1)[:, ::-1]
    assert ((GS[:, 0] - GS[:, 1]) > 1e-3).all()
    b = O.layer_backward(f, w13, w2, dy, with_aux=True)
    rng = np.random.default_rng(6)
    h = 1e-6

    def loss_at(x_, w_r_, w13_, w2_):
        f_ = O.layer_forward(cfg, x_, w_r_, w13_, w2_)
        assert (f_["expert_idx"] == f["expert_idx"]).all()
        return O.layer_loss(f_, dy)

    for name in ("x", "w_r", "w13_0", "w13_1", "w2_0", "w2_1"):
        for trial in range(3):
            params = dict(x=x, w_r=w_r, w13_0=w13[0], w13_1=w13[1], w2_0=w2[0], w2_1=w2[1])
            grads = dict(x=b["dx"], w_r=b["dw_r"], w13_0=b["dw13"][0], w13_1=b["dw13"][1],
                         w2_0=b["dw2"][0], w2_1=b["dw2"][1])
            v = rng.normal(size=params[name].shape)

            def shifted(s):
                p = dict(params)
                p[name] = params[name] + s * h * v
                return loss_at(p["x"], p["w_r"], [p["w13_0"], p["w13_1"]], [p["w2_0"], p["w2_1"]])

            fd = (shifted(+1) - shifted(-1)) / (2 * h)
            an = float(np.sum(grads[name] * v))
            assert abs(fd - an) <= 1e-6 * max(1.0, abs(an)), (name, fd, an)


def test_sampled_tokens_reproduce_full_batch_rows():
    # y_t and dx_t depend on token t alone once the batch statistics are handed over
    cfg = O.OracleConfig(d_model=8, n_groups=2, experts_per_group=4, k_groups=1, k_experts=2,
                         group_width=[12, 6], alpha_g=0.3, alpha_e=0.4)
    T = 50
    x, w_r, w13, w2, dy = _rand_layer(cfg, T, 9)
    f = O.layer_forward(cfg, x, w_r, w13, w2)
    b = O.layer_backward(f, w13, w2, dy)
    samp = np.array([3, 17, 18, 44])
    fs = O.layer_forward(cfg, x[samp], w_r, w13, w2)
    bs = O.layer_backward(fs, w13, w2, dy[samp],
                          aux_counts=(f["stats"]["cG"], f["stats"]["cE_lit"], T))
    np.testing.assert_allclose(fs["y"], f["y"][samp], rtol=1e-13)
    np.testing.assert_allclose(bs["dx"], b["dx"][samp], rtol=1e-12, atol=1e-14)


def test_shared_experts_add_an_ungated_dense_ffn_and_its_gradients():
    # N_s shared FFNs of width W, weights concatenated along the hidden axis, applied to every
    # token: autograd of (independent dense routed forward + three-line dense FFN) must agree
    cfg = O.OracleConfig(d_model=10, n_groups=2, experts_per_group=3, k_groups=1, k_experts=2,
                         group_width=[8, 12], alpha_g=0.7, alpha_e=0.9)
    T, Ws, Ns = 30, 6, 2
    x, w_r, w13, w2, dy = _rand_layer(cfg, T, 33)
    rng = np.random.default_rng(34)
    sh_g = [rng.normal(size=(Ws, 10)) * 0.3 for _ in range(Ns)]      # per shared expert
    sh_u = [rng.normal(size=(Ws, 10)) * 0.3 for _ in range(Ns)]
    sh_d = [rng.normal(size=(10, Ws)) * 0.3 for _ in range(Ns)]
    w13_s = np.concatenate(sh_g + sh_u, axis=0)                       # [2 * Ns * Ws, d]
    w2_s = np.concatenate(sh_d, axis=1)                               # [d, Ns * Ws]
    f = O.layer_forward(cfg, x, w_r, w13, w2, shared=(w13_s, w2_s))
    b = O.layer_backward(f, w13, w2, dy, shared=(w13_s, w2_s))
    f0 = O.layer_forward(cfg, x, w_r, w13, w2)
    # forward: the sum of the N_s separate FFNs
    extra = sum((torch.nn.functional.silu(torch.tensor(x) @ torch.tensor(g_).T)
                 * (torch.tensor(x) @ torch.tensor(u_).T)) @ torch.tensor(d_).T
                for g_, u_, d_ in zip(sh_g, sh_u, sh_d)).numpy()
    np.testing.assert_allclose(f["y"], f0["y"] + extra, rtol=1e-11, atol=1e-12)
    # backward: autograd of routed + shared
    tx = torch.tensor(x, requires_grad=True)
    twr = torch.tensor(w_r, requires_grad=True)
    tw13 = [torch.tensor(w, requires_grad=True) for w in w13]
    tw2 = [torch.tensor(w, requires_grad=True) for w in w2]
    t13s, t2s = torch.tensor(w13_s, requires_grad=True), torch.tensor(w2_s, requires_grad=True)
    H = Ns * Ws
    _, loss, _, _ = _torch_dense_forward(cfg, tx, twr, tw13, tw2, torch.tensor(dy))
    ys = (torch.nn.functional.silu(tx @ t13s[:H].T) * (tx @ t13s[H:].T)) @ t2s.T
    (loss + torch.sum(ys * torch.tensor(dy))).backward()
    tol = dict(rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose(b["dx"], tx.grad.numpy(), **tol)
    np.testing.assert_allclose(b["dw_r"], twr.grad.numpy(), **tol)
    np.testing.assert_allclose(b["shared"]["dw13"], t13s.grad.numpy(), **tol)
    np.testing.assert_allclose(b["shared"]["dw2"], t2s.grad.numpy(), **tol)
    for g in range(2):
        np.testing.assert_allclose(b["dw13"][g], tw13[g].grad.numpy(), **tol)
