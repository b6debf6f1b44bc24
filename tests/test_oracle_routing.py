"""Pins for the oracle's router (Eq. 2-6): brute force, closed forms, library
special cases, invariants, and the float32 selection contract."""
import itertools
import math

import numpy as np
import pytest
from scipy.special import softmax as sp_softmax

import oracle as O


def _cfg(N_g=2, N=4, K_g=1, K_e=2, widths=None, **kw):
    widths = widths or [64 * (g + 1) for g in range(N_g)]
    return O.OracleConfig(d_model=16, n_groups=N_g, experts_per_group=N, k_groups=K_g,
                          k_experts=K_e, group_width=widths, **kw)


def _best_subset(keys, K, allowed=None):
    """The size-K index set whose descending key tuple is lexicographically
    largest; among equals the lexicographically smallest index tuple.  Returned
    in slot order (descending key, ties by index)."""
    idx = [i for i in range(len(keys)) if allowed is None or allowed[i]]
    best = None
    for sub in itertools.combinations(idx, K):
        order = sorted(sub, key=lambda i: (-keys[i], i))
        sig = (tuple(-keys[i] for i in order), tuple(sorted(sub)))
        if best is None or sig < best[0]:
            best = (sig, order)
    return best[1]


def _brute_route(cfg, logit_row):
    N_g, N = cfg.n_groups, cfg.experts_per_group
    GS = [1.0 / (1.0 + math.exp(-v)) for v in logit_row[:N_g]]
    groups = _best_subset(GS, cfg.k_groups)
    ESpp = [0.0] * (N_g * N)
    allowed = [False] * (N_g * N)
    for g in groups:
        l = logit_row[N_g + g * N: N_g + (g + 1) * N]
        m = max(l)
        ex = [math.exp(v - m) for v in l]
        s = sum(ex)
        for i in range(N):
            ESpp[g * N + i] = ex[i] / s * GS[g]
            allowed[g * N + i] = True
    experts = _best_subset(ESpp, cfg.k_experts, allowed)
    tot = sum(ESpp[e] for e in experts)
    gate = [ESpp[e] / tot for e in experts]
    return groups, experts, gate


@pytest.mark.parametrize("N_g,N,K_g,K_e", [(2, 4, 1, 2), (2, 4, 2, 3), (3, 2, 2, 4), (2, 3, 2, 2),
                                             (4, 2, 3, 5), (1, 6, 1, 3)])
def test_route_definition_matches_brute_force(N_g, N, K_g, K_e):
    cfg = _cfg(N_g, N, K_g, K_e)
    rng = np.random.default_rng(N_g * 100 + N * 10 + K_e)
    T = 60
    logits = rng.normal(size=(T, N_g + N_g * N))
    # deliberate ties: quantised logits on a third of the rows, all-equal rows too
    logits[:20] = np.round(logits[:20])
    logits[20:24] = 0.5
    r = O.route_definition(cfg, logits)
    for t in range(T):
        groups, experts, gate = _brute_route(cfg, list(logits[t]))
        assert list(r["group_idx"][t]) == groups, t
        assert list(r["expert_idx"][t]) == experts, t
        np.testing.assert_allclose(r["gate"][t], gate, rtol=1e-13)


def test_zero_router_closed_form():
    # every logit 0 => GS = 1/2, ES' = 1/N, all keys tie => lowest indices win
    cfg = _cfg(N_g=3, N=4, K_g=2, K_e=6)
    T = 5
    r = O.route_definition(cfg, np.zeros((T, 3 + 12)))
    assert (r["group_idx"] == np.array([0, 1])).all()
    assert (r["expert_idx"] == np.arange(6)).all()          # group 0 fills up, spills into group 1
    np.testing.assert_allclose(r["gate"], 1.0 / 6, rtol=1e-15)
    np.testing.assert_allclose(r["GS"], 0.5)
    np.testing.assert_allclose(r["ESp"][:, :8], 0.25)
    assert (r["ESp"][:, 8:] == 0).all()
    s = O.route_spec(cfg, np.zeros((T, 15), np.float32))
    assert (s["group_idx"] == r["group_idx"]).all() and (s["expert_idx"] == r["expert_idx"]).all()
    np.testing.assert_allclose(s["gate"], 1.0 / 6, rtol=1e-6)


def test_single_group_is_textbook_softmax_topk_renormalise():
    # N_g = K_g = 1: GS cancels in Eq. 6 -> softmax, top-k, renormalise.
    cfg = _cfg(N_g=1, N=8, K_g=1, K_e=3)
    rng = np.random.default_rng(3)
    logits = rng.normal(size=(200, 9)) * 2
    r = O.route_definition(cfg, logits)
    p = sp_softmax(logits[:, 1:], axis=1)
    idx = np.argsort(-p, axis=1, kind="stable")[:, :3]
    sel = np.take_along_axis(p, idx, axis=1)
    assert (r["expert_idx"] == idx).all()
    np.testing.assert_allclose(r["gate"], sel / sel.sum(1, keepdims=True), rtol=1e-12)


def test_select_everything_is_dense_mixture():
    cfg = _cfg(N_g=2, N=3, K_g=2, K_e=6)
    rng = np.random.default_rng(4)
    logits = rng.normal(size=(50, 8))
    r = O.route_definition(cfg, logits)
    GS = 1 / (1 + np.exp(-logits[:, :2]))
    es = np.concatenate([sp_softmax(logits[:, 2:5], axis=1) * GS[:, :1],
                         sp_softmax(logits[:, 5:8], axis=1) * GS[:, 1:]], axis=1)
    dense = es / es.sum(1, keepdims=True)
    got = np.zeros_like(dense)
    np.put_along_axis(got, r["expert_idx"].astype(np.int64), r["gate"], axis=1)
    np.testing.assert_allclose(got, dense, rtol=1e-12)


@pytest.mark.parametrize("N_g,N,K_g,K_e", [(3, 8, 2, 4), (4, 16, 2, 6), (8, 4, 3, 6)])
def test_routing_invariants(N_g, N, K_g, K_e):
    cfg = _cfg(N_g, N, K_g, K_e)
    rng = np.random.default_rng(5)
    T = 300
    logits = rng.normal(size=(T, N_g + N_g * N))
    r = O.route_definition(cfg, logits)
    np.testing.assert_allclose(r["gate"].sum(1), 1.0, rtol=1e-13)              # Eq. 6
    esp = r["ESp"].reshape(T, N_g, N).sum(2)
    np.testing.assert_allclose(esp[r["group_mask"]], 1.0, rtol=1e-13)          # Eq. 3, selected
    assert (esp[~r["group_mask"]] == 0).all()                                  # Eq. 3, otherwise
    assert (r["group_mask"].sum(1) == K_g).all()
    for t in range(T):
        assert len(set(r["expert_idx"][t])) == K_e
        assert set(r["expert_idx"][t] // N) <= set(r["group_idx"][t])          # experts inside chosen groups
    # gate proportional to ES'' on the selected set, slots in descending order
    key = np.take_along_axis(r["ESpp"], r["expert_idx"].astype(np.int64), axis=1)
    assert (np.diff(key, axis=1) <= 0).all()
    np.testing.assert_allclose(r["gate"] * key.sum(1, keepdims=True), key, rtol=1e-13)


# ---------------- float32 selection contract ----------------

def _ulp32(x):
    return np.spacing(np.float32(abs(x)))


def test_exp_spec_within_two_ulp_of_libm():
    z = np.concatenate([-np.linspace(0, 87, 20001), -np.logspace(-8, 1.9, 5000)]).astype(np.float32)
    got = O.exp_spec(z).astype(np.float64)
    ref = np.exp(z.astype(np.float64))
    ulp = np.spacing(ref.astype(np.float32)).astype(np.float64)
    assert np.max(np.abs(got - ref) / ulp) <= 2.0
    assert O.exp_spec(np.float32(0.0)) == np.float32(1.0)
    assert O.exp_spec(np.float32(-87.5)) == 0 and O.exp_spec(np.float32(-1e30)) == 0


def test_sigmoid_spec_close_to_definition():
    z = np.linspace(-30, 30, 6001).astype(np.float32)
    got = O.sigmoid_spec(z).astype(np.float64)
    ref = 1 / (1 + np.exp(-z.astype(np.float64)))
    assert np.max(np.abs(got - ref) / ref) < 4e-7
    assert O.sigmoid_spec(np.float32(0)) == np.float32(0.5)


def test_tree_sum_order():
    p = np.array([1e8, 1.0, -1e8, 1.0, 3.0], np.float32)
    # ((1e8+1)+(-1e8+1)) + ((3+0)+(0+0)) in float32
    f = np.float32
    want = f(f(f(p[0] + p[1]) + f(p[2] + p[3])) + f(f(p[4] + f(0)) + f(0)))
    assert O.tree_sum_f32(p) == want


def test_spec_matches_definition_off_the_fragile_set():
    cfg = _cfg(4, 16, 2, 6)
    rng = np.random.default_rng(7)
    T = 4000
    logits = (rng.normal(size=(T, 4 + 64)) * 0.9).astype(np.float32)
    d = O.route_definition(cfg, logits.astype(np.float64))
    s = O.route_spec(cfg, logits)
    # margin between the K-th and (K+1)-th key on both levels (fp64)
    GS = np.sort(d["GS"], axis=1)[:, ::-1]
    mg = (GS[:, 1] - GS[:, 2]) / GS[:, 1]
    keys = np.sort(np.where(np.repeat(d["group_mask"], 16, 1), d["ESpp"], -1.0), axis=1)[:, ::-1]
    me = (keys[:, 5] - keys[:, 6]) / keys[:, 5]
    safe = (mg > 1e-4) & (me > 1e-4)
    assert safe.mean() > 0.99
    assert (d["group_idx"][safe] == s["group_idx"][safe]).all()
    # the selected SET is fixed by the margin; slot order may differ on near-equal keys
    assert (np.sort(d["expert_idx"][safe], 1) == np.sort(s["expert_idx"][safe], 1)).all()
    same = (d["expert_idx"] == s["expert_idx"]).all(1)
    np.testing.assert_allclose(s["gate"][same], d["gate"][same], rtol=2e-6)
    np.testing.assert_allclose(s["ESp"], d["ESp"], rtol=2e-6, atol=1e-12)
    np.testing.assert_allclose(s["GS"], d["GS"], rtol=1e-6)


def test_spec_tie_breaks_and_group_order():
    cfg = _cfg(N_g=4, N=4, K_g=2, K_e=5)
    lg = np.zeros((3, 4 + 16), np.float32)
    lg[1, :4] = [0.0, 1.0, 1.0, -0.0]       # groups 1,2 tie -> 1 then 2
    lg[2, :4] = [-0.0, 0.0, -1.0, -2.0]     # +0 and -0 compare equal -> 0 then 1
    s = O.route_spec(cfg, lg)
    assert list(s["group_idx"][0]) == [0, 1]
    assert list(s["group_idx"][1]) == [1, 2]
    assert list(s["group_idx"][2]) == [0, 1]
    assert list(s["expert_idx"][0]) == [0, 1, 2, 3, 4]
    assert list(s["expert_idx"][1]) == [4, 5, 6, 7, 8]


def test_nan_logits_rank_below_every_number():
    """Reading of Eq. 2-5 for NaN scores (the paper orders real numbers only): a NaN logit loses
    against every number, ties among NaNs go to the lowest index, and the entries are counted.
    Pinned without route_spec's own arithmetic: the selections must equal those of the same
    logits with every NaN replaced by a number far below all others, and an all-NaN token must
    select what the all-equal (zero) token selects."""
    cfg = O.OracleConfig(d_model=8, n_groups=3, experts_per_group=4, k_groups=2, k_experts=5,
                         group_width=[8, 8, 8])
    rng = np.random.default_rng(5)
    lg = rng.normal(size=(64, 3 + 12)).astype(np.float32)
    nan_at = rng.random(lg.shape) < 0.2
    nan_at[0] = True                                   # one token with nothing but NaN
    nan_at[1, :3] = True                               # all group logits NaN
    nan_at[2, 3:7] = True                              # a whole group of expert logits NaN
    with_nan = np.where(nan_at, np.nan, lg).astype(np.float32)
    very_low = np.where(nan_at, -1e30, lg).astype(np.float32)
    a, b = O.route_spec(cfg, with_nan), O.route_spec(cfg, very_low)
    assert a["nan_logits"] == int(nan_at.sum()) and b["nan_logits"] == 0
    assert (a["group_idx"] == b["group_idx"]).all() and (a["expert_idx"] == b["expert_idx"]).all()
    zero = O.route_spec(cfg, np.zeros((1, 15), np.float32))
    assert (a["group_idx"][0] == zero["group_idx"][0]).all()
    assert (a["expert_idx"][0] == zero["expert_idx"][0]).all()
    # gates stay a convex combination wherever the chosen groups have numbers for logits (a NaN
    # group logit has sigmoid 0, so a token whose chosen groups are all NaN has only zero keys)
    ok = ~nan_at[:, :3].any(axis=1)
    assert np.isfinite(a["gate"][ok]).all() and np.allclose(a["gate"][ok].sum(axis=1), 1.0, atol=1e-6)
    # a NaN expert is only ever picked when fewer than K_e numbers are on offer in the chosen groups
    picked_nan = np.take_along_axis(nan_at[:, 3:], a["expert_idx"].astype(np.int64), axis=1)
    for t in np.nonzero(ok)[0]:
        chosen = a["group_idx"][t]
        numbers = sum(int((~nan_at[t, 3 + 4 * g:3 + 4 * g + 4]).sum()) for g in chosen)
        assert int(picked_nan[t].sum()) == max(0, cfg.k_experts - numbers)
