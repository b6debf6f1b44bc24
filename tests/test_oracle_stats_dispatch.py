"""Pins for the oracle's auxiliary statistics (Eq. 7-14) and token permutation."""
import numpy as np
import pytest

import oracle as O


def _cfg(N_g, N, K_g, K_e, widths=None, **kw):
    widths = widths or [64 * (g + 1) for g in range(N_g)]
    return O.OracleConfig(d_model=16, n_groups=N_g, experts_per_group=N, k_groups=K_g,
                          k_experts=K_e, group_width=widths, **kw)


def test_zero_router_losses_closed_form():
    # GS = 1/2 everywhere -> s' = 1/N_g, p^G = 1/N_g; groups 0..K_g-1 chosen by every token:
    # f^G_g = (N_g/K_g) T (1/T) -> L_G = alpha_G/K_g * sum_{g<K_g} W_g/W_max.
    cfg = _cfg(3, 4, 2, 6, widths=[100, 200, 400])
    T = 17
    r = O.route_definition(cfg, np.zeros((T, 15)))
    st = O.aux_stats(cfg, r["GS"], r["ESp"], r["group_idx"], r["expert_idx"])
    assert list(st["cG"]) == [T, T, 0]
    np.testing.assert_allclose(st["sG"], T / 3)
    want_LG = cfg.alpha_g / 2 * (100 / 400 + 200 / 400)
    np.testing.assert_allclose(st["L_G"], want_LG, rtol=1e-13)
    # ES' = 1/4 on 8 experts, 0 on the rest; literal indicator picks experts 0..5 (ties -> lowest)
    assert list(st["cE_lit"]) == [T] * 6 + [0] * 6
    assert list(st["cE_route"]) == [T] * 6 + [0] * 6
    np.testing.assert_allclose(st["sE"][:8], T * 0.25 / (1 + 1e-20))
    assert (st["sE"][8:] == 0).all()
    # L_E = alpha_E * sum_e f_e p_e,  f_e = (N/K_e) T / T = 4/6 for e<6,  p_e = 1/4
    np.testing.assert_allclose(st["L_E"], cfg.alpha_e * 6 * (4 / 6) * 0.25, rtol=1e-13)
    # literal Eq. 8 / Eq. 12 (no 1/T in f) scales both losses by T
    cfg2 = _cfg(3, 4, 2, 6, widths=[100, 200, 400], f_norm_by_T=False)
    st2 = O.aux_stats(cfg2, r["GS"], r["ESp"], r["group_idx"], r["expert_idx"])
    np.testing.assert_allclose(st2["L_G"], want_LG * T, rtol=1e-13)
    np.testing.assert_allclose(st2["L_E"], st["L_E"] * T, rtol=1e-13)


@pytest.mark.parametrize("N_g,N,K_g,K_e", [(3, 8, 2, 4), (4, 16, 2, 6), (8, 4, 3, 6)])
def test_stats_invariants_and_naive_recount(N_g, N, K_g, K_e):
    cfg = _cfg(N_g, N, K_g, K_e)
    rng = np.random.default_rng(11)
    T = 257
    logits = rng.normal(size=(T, N_g + N_g * N))
    r = O.route_definition(cfg, logits)
    st = O.aux_stats(cfg, r["GS"], r["ESp"], r["group_idx"], r["expert_idx"])
    assert st["cG"].sum() == T * K_g
    assert st["cE_route"].sum() == T * K_e and st["cE_lit"].sum() == T * K_e
    np.testing.assert_allclose(st["sG"].sum(), T, rtol=1e-12)                  # Eq. 10 sums to one
    np.testing.assert_allclose(st["sE"].sum(), T * K_g / (1 + cfg.eps), rtol=1e-12)
    # naive O(T*N_e) recount with python loops, straight from the indicator definitions
    cG = [0] * N_g
    cE = [0] * (N_g * N)
    cL = [0] * (N_g * N)
    sG = np.zeros(N_g)
    sE = np.zeros(N_g * N)
    for t in range(T):
        gs = 1 / (1 + np.exp(-logits[t, :N_g]))
        order = sorted(range(N_g), key=lambda g: (-gs[g], g))[:K_g]
        for g in order:
            cG[g] += 1
        sG += gs / gs.sum()
        esp = np.zeros(N_g * N)
        for g in order:
            l = logits[t, N_g + g * N:N_g + (g + 1) * N]
            p = np.exp(l - l.max())
            esp[g * N:(g + 1) * N] = p / p.sum()
        espp = esp * np.repeat(gs, N)
        allowed = [e for e in range(N_g * N) if e // N in order]
        for e in sorted(allowed, key=lambda e: (-espp[e], e))[:K_e]:
            cE[e] += 1
        for e in sorted(allowed, key=lambda e: (-esp[e], e))[:K_e]:
            cL[e] += 1
        for g in range(N_g):
            seg = esp[g * N:(g + 1) * N]
            sE[g * N:(g + 1) * N] += seg / (seg.sum() + cfg.eps)
    assert list(st["cG"]) == cG and list(st["cE_route"]) == cE and list(st["cE_lit"]) == cL
    np.testing.assert_allclose(st["sG"], sG, rtol=1e-12)
    np.testing.assert_allclose(st["sE"], sE, rtol=1e-12)
    # losses from the raw sums, Eq. 7 and Eq. 11 typed out
    W = np.array(cfg.group_width, float)
    LG = cfg.alpha_g * sum(W[g] / W.max() * (N_g / K_g * cG[g] / T) * (sG[g] / T) for g in range(N_g))
    LE = cfg.alpha_e * sum((N / K_e * cL[e] / T) * (sE[e] / T) for e in range(N_g * N))
    np.testing.assert_allclose(st["L_G"], LG, rtol=1e-12)
    np.testing.assert_allclose(st["L_E"], LE, rtol=1e-12)
    # fe_mode 1 uses the routing mask instead
    cfg1 = _cfg(N_g, N, K_g, K_e, fe_mode=1)
    st1 = O.aux_stats(cfg1, r["GS"], r["ESp"], r["group_idx"], r["expert_idx"])
    LE1 = cfg.alpha_e * sum((N / K_e * cE[e] / T) * (sE[e] / T) for e in range(N_g * N))
    np.testing.assert_allclose(st1["L_E"], LE1, rtol=1e-12)


@pytest.mark.parametrize("align", [1, 8, 128])
def test_dispatch_algebra(align):
    rng = np.random.default_rng(2)
    T, K, N_e = 333, 3, 10
    expert_idx = np.stack([rng.permutation(N_e)[:K] for _ in range(T)]).astype(np.int32)
    expert_idx[:, :] = np.where(expert_idx == 9, 8, expert_idx)                # expert 9 gets nothing
    # rows with a duplicated expert are not valid routing output; rebuild those rows
    for t in range(T):
        while len(set(expert_idx[t])) < K:
            expert_idx[t] = rng.permutation(9)[:K]
    dp = O.dispatch(expert_idx, N_e, align)
    R = T * K
    assert dp["counts"].sum() == R and dp["counts"][9] == 0
    assert (dp["offsets"] == np.concatenate([[0], np.cumsum(dp["counts"])])).all()
    assert sorted(dp["row_of"].ravel()) == list(range(R))                       # bijection onto [0, R)
    assert (dp["src_of"][dp["row_of"].ravel()] == np.arange(R)).all()           # src_of inverts row_of
    for e in range(N_e):
        rows = np.arange(dp["offsets"][e], dp["offsets"][e + 1])
        src = dp["src_of"][rows]
        assert (expert_idx.ravel()[src] == e).all()
        assert (np.diff(src // K) > 0).all() if len(src) > 1 else True          # ascending token order
    assert (dp["aligned_offsets"] % align == 0).all()
    seg = np.diff(dp["aligned_offsets"])
    assert ((seg >= dp["counts"]) & (seg < dp["counts"] + align)).all()
    e_of = expert_idx
    assert (dp["prow_of"] - dp["aligned_offsets"][e_of] == dp["row_of"] - dp["offsets"][e_of]).all()
    # permute then un-permute (unit gates, any one slot) gives x back bit for bit
    x = rng.normal(size=(T, 5)).astype(np.float32)
    xp = O.permute_rows(x, dp["prow_of"], int(dp["aligned_offsets"][-1]))
    for k in range(K):
        assert (xp[dp["prow_of"][:, k]] == x).all()
    used = np.zeros(xp.shape[0], bool)
    used[dp["prow_of"].ravel()] = True
    assert (xp[~used] == 0).all()
