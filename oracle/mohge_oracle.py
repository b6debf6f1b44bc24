"""fp64 CPU oracle of the MoHGE expert layer (forward and backward).

TEST INFRASTRUCTURE ONLY: imported by the test-suite, by the smoke check and by
the benchmark's CPU-baseline leg. It shares no code, table or constant
generator with the CUDA library and must never be reachable from the product
path.

Everything here is the paper's definition written out with plain numpy in
float64 (Sec. 3.1-3.4, Eq. 2-14, and the layer output in the form of Eq. 15 of
the appendix).  A matmul is used as a library step; there is no blocking,
fusion or reordering.  One extra routing mode ("spec") evaluates the selection
in a fully specified float32 arithmetic so that integer outputs of an
independent float32 implementation can be compared bit for bit.

Notation (paper): T tokens, N_g groups, N experts per group, N_e = N_g*N
experts, K_g groups per token, K_e experts per token, W_g hidden width of
group g.  Flat expert id e = g*N + i.  Router weight rows: first the N_g group
centroids e_g (Eq. 2), then the N_e expert embeddings e_{g,i} (Eq. 3),
group-major.

Readings taken where the paper is silent (each also listed in the design
notes): experts are bias-free SwiGLU FFNs; the layer output is the gate-weighted
sum over the selected experts only; "topK" picks exactly K entries with ties
going to the lowest index; experts of unselected groups can never be picked by
Eq. 5; Eq. 9 and Eq. 13 sum over tokens t = 1..T.

Pin status: every function below is pinned by tests/test_oracle_*.py (brute
force, closed forms, invariants, library special cases, finite differences,
autograd of an independently written forward).  Nothing is "parity unpinned".
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

import numpy as np

__all__ = [
    "OracleConfig", "router_logits", "topk_rounds", "route_definition",
    "route_values", "gates_from_selection", "exp_spec", "sigmoid_spec",
    "tree_sum_f32", "route_spec", "aux_stats", "dispatch", "permute_rows",
    "swiglu_ffn", "expert_backward", "layer_forward", "layer_backward", "layer_loss",
    "aux_losses",
]


@dataclass
class OracleConfig:
    d_model: int
    n_groups: int                 # N_g
    experts_per_group: int        # N
    k_groups: int                 # K_g
    k_experts: int                # K_e
    group_width: Sequence[int]    # W_g, one per group
    alpha_g: float = 1e-4         # Table 8 optimum
    alpha_e: float = 2.5e-3       # Table 8 optimum
    eps: float = 1e-20            # Eq. 14
    f_norm_by_T: bool = True      # f^G, f^E carry a 1/T ("normalized routing frequency")
    fe_mode: int = 0              # 0: Eq. 12 literally (top-K_e of ES'); 1: the actual routing mask

    @property
    def n_experts(self) -> int:
        return self.n_groups * self.experts_per_group

    def check(self) -> None:
        assert len(self.group_width) == self.n_groups
        assert 1 <= self.k_groups <= self.n_groups
        assert 1 <= self.k_experts <= self.k_groups * self.experts_per_group


# --------------------------------------------------------------------------
# Router (Sec. 3.2)
# --------------------------------------------------------------------------

def router_logits(x, w_r, logit_bias=None):
    """Arguments of Eq. 2 and Eq. 3: x_t . e_g and x_t . e_{g,i}  ->  [T, N_g+N_e]."""
    logits = np.asarray(x, np.float64) @ np.asarray(w_r, np.float64).T
    if logit_bias is not None:
        logits = logits + np.asarray(logit_bias, np.float64)[None, :]
    return logits


def topk_rounds(keys, K):
    """Exactly K picks per row: K rounds of arg-max, ties to the lowest index.

    Slot k holds the k-th largest key (Eq. 2 text "the K_g groups with the
    highest scores", Eq. 5)."""
    keys = np.array(keys, copy=True)
    T = keys.shape[0]
    idx = np.empty((T, K), np.int32)
    rows = np.arange(T)
    for k in range(K):
        j = np.argmax(keys, axis=1)          # first maximum = lowest index
        idx[:, k] = j
        keys[rows, j] = -np.inf
    return idx


def route_values(cfg: OracleConfig, logits, group_idx):
    """GS (Eq. 2), ES' (Eq. 3) and ES'' (Eq. 4) in fp64 for a given group selection."""
    N_g, N = cfg.n_groups, cfg.experts_per_group
    logits = np.asarray(logits, np.float64)
    T = logits.shape[0]
    lG = logits[:, :N_g]
    lE = logits[:, N_g:].reshape(T, N_g, N)
    GS = 1.0 / (1.0 + np.exp(-lG))                                  # Eq. 2
    gsel = np.zeros((T, N_g), bool)
    gsel[np.arange(T)[:, None], group_idx] = True
    m = lE.max(axis=2, keepdims=True)
    p = np.exp(lE - m)
    ESp = p / p.sum(axis=2, keepdims=True)                          # group-wise softmax
    ESp = np.where(gsel[:, :, None], ESp, 0.0)                      # Eq. 3
    ESpp = ESp * GS[:, :, None]                                     # Eq. 4
    return dict(GS=GS, ESp=ESp.reshape(T, N_g * N), ESpp=ESpp.reshape(T, N_g * N),
                group_mask=gsel)


def gates_from_selection(ESpp, expert_idx):
    """Eq. 5 + Eq. 6: keep the selected ES'' and normalise them to sum to one."""
    key = np.take_along_axis(ESpp, expert_idx.astype(np.int64), axis=1)
    return key / key.sum(axis=1, keepdims=True)


def route_definition(cfg: OracleConfig, logits):
    """Two-level routing exactly as Eq. 2-6, float64 throughout."""
    cfg.check()
    N_g, N = cfg.n_groups, cfg.experts_per_group
    logits = np.asarray(logits, np.float64)
    GS_all = 1.0 / (1.0 + np.exp(-logits[:, :N_g]))
    group_idx = topk_rounds(GS_all, cfg.k_groups)                   # top-K_g of GS_t
    v = route_values(cfg, logits, group_idx)
    sel_e = np.repeat(v["group_mask"], N, axis=1)
    keys = np.where(sel_e, v["ESpp"], -1.0)                         # unselected groups cannot win
    expert_idx = topk_rounds(keys, cfg.k_experts)                   # Eq. 5
    gate = gates_from_selection(v["ESpp"], expert_idx)              # Eq. 6
    return dict(group_idx=group_idx, expert_idx=expert_idx, gate=gate, **v)


# ---- float32 "spec" arithmetic: the selection contract --------------------
#
# All operations are IEEE-754 binary32, round-to-nearest-even, one rounding per
# written operation, no fused multiply-add, subnormals kept.

_F = np.float32
_LOG2E = _F(float.fromhex("0x1.715476p+0"))
_LN2_HI = _F(float.fromhex("0x1.62e4p-1"))
_LN2_LO = _F(float.fromhex("0x1.7f7d1cp-20"))
_EXP_C = [_F(float.fromhex(h)) for h in (
    "0x1.a01a02p-13",   # 1/7!
    "0x1.6c16c2p-10",   # 1/6!
    "0x1.111112p-7",    # 1/5!
    "0x1.555556p-5",    # 1/4!
    "0x1.555556p-3",    # 1/3!
    "0x1p-1",           # 1/2!
    "0x1p+0",
    "0x1p+0",
)]


def exp_spec(z):
    """float32 exp for z <= 0: range reduction by ln2 (two-piece), degree-7
    Taylor polynomial in Horner form with separate multiply and add, exact
    scaling by 2^n; z < -87 gives +0."""
    z_in = np.asarray(z, dtype=_F)
    z = np.maximum(z_in, _F(-100.0))          # values below -87 are replaced by +0 at the end
    n = np.rint(z * _LOG2E).astype(_F)
    r = z - n * _LN2_HI
    r = r - n * _LN2_LO
    p = np.full_like(r, _EXP_C[0])
    for c in _EXP_C[1:]:
        p = p * r + c
    n_i = np.clip(n.astype(np.int32), -126, 0)
    scale = ((n_i + 127) << 23).astype(np.int32).view(_F)
    out = p * scale
    return np.where(z_in < _F(-87.0), _F(0.0), out).astype(_F)


def sigmoid_spec(z):
    z = np.asarray(z, dtype=_F)
    e = exp_spec(-np.abs(z))
    one = _F(1.0)
    return np.where(z >= 0, one / (one + e), e / (one + e)).astype(_F)


def tree_sum_f32(p):
    """Balanced binary tree sum over the last axis (padded with +0 to a power
    of two): level by level, neighbours (2j, 2j+1) are added."""
    p = np.asarray(p, dtype=_F)
    n = p.shape[-1]
    P = 1
    while P < n:
        P *= 2
    if P != n:
        pad = np.zeros(p.shape[:-1] + (P - n,), _F)
        p = np.concatenate([p, pad], axis=-1)
    while p.shape[-1] > 1:
        p = (p[..., 0::2] + p[..., 1::2]).astype(_F)
    return p[..., 0]


def route_spec(cfg: OracleConfig, logits32):
    """Selection contract in float32.

    Groups: K_g rounds of arg-max over the raw group logits (sigmoid is
    monotone).  For a selected group: p_i = exp_spec(l_i - max_i l_i),
    S = tree sum of p, r = sigmoid_spec(l_g)/S, key_i = p_i * r, ES'_i = p_i/S.
    Experts of unselected groups get key -1.  Experts: K_e rounds of arg-max
    over the keys.  gate_k = key_k / (left-to-right sum of the K_e keys).

    NaN logits: Eq. 2-5 order real numbers and say nothing about NaN.  Reading:
    a NaN logit is invalid input that ranks below every number; it is read as
    the most negative finite float32, ties among such entries go to the lowest
    index as everywhere else, and the number of NaN entries is returned in
    "nan_logits" (an implementation reports them through its status word).
    """
    cfg.check()
    N_g, N = cfg.n_groups, cfg.experts_per_group
    logits32 = np.asarray(logits32, dtype=_F)
    nan_logits = int(np.isnan(logits32).sum())
    if nan_logits:
        logits32 = np.where(np.isnan(logits32), -np.finfo(_F).max, logits32).astype(_F)
    T = logits32.shape[0]
    lG = logits32[:, :N_g]
    lE = logits32[:, N_g:].reshape(T, N_g, N)
    group_idx = topk_rounds(lG, cfg.k_groups)
    gsel = np.zeros((T, N_g), bool)
    gsel[np.arange(T)[:, None], group_idx] = True
    GS = sigmoid_spec(lG)
    m = lE.max(axis=2, keepdims=True)
    with np.errstate(over="ignore"):                      # -FLT_MAX - m may round to -inf: exp gives 0
        p = exp_spec((lE - m).astype(_F))
    S = tree_sum_f32(p)                                   # [T, N_g]
    r = (GS / S).astype(_F)
    key = (p * r[:, :, None]).astype(_F)
    ESp = (p / S[:, :, None]).astype(_F)
    key = np.where(gsel[:, :, None], key, _F(-1.0)).reshape(T, N_g * N)
    ESp = np.where(gsel[:, :, None], ESp, _F(0.0)).reshape(T, N_g * N)
    expert_idx = topk_rounds(key, cfg.k_experts)
    ksel = np.take_along_axis(key, expert_idx.astype(np.int64), axis=1)
    ssum = ksel[:, 0].copy()
    for k in range(1, cfg.k_experts):
        ssum = (ssum + ksel[:, k]).astype(_F)
    with np.errstate(invalid="ignore"):                   # all keys 0 (chosen groups all NaN): 0/0
        gate = (ksel / ssum[:, None]).astype(_F)
    return dict(group_idx=group_idx, expert_idx=expert_idx, gate=gate, GS=GS,
                ESp=ESp, key=key, group_mask=gsel, nan_logits=nan_logits)


# --------------------------------------------------------------------------
# Auxiliary-loss statistics (Sec. 3.3 Eq. 7-10, Sec. 3.4.2 Eq. 11-14)
# --------------------------------------------------------------------------

def aux_stats(cfg: OracleConfig, GS, ESp, group_idx, expert_idx, esp_keys=None):
    """Counts and score sums behind L_G and L_E, and the two loss values.

    cG[g]        number of tokens whose top-K_g contains g          (indicator of Eq. 8)
    sG[g]        sum_t GS_{g,t} / sum_j GS_{j,t}                    (Eq. 9-10)
    cE_route[e]  number of tokens routed to e (Eq. 5 selection)
    cE_lit[e]    number of tokens with ES'_{e,t} in top-K_e(ES'_t)  (indicator of Eq. 12)
    sE[e]        sum_t ES'_{e,t} / (sum_{j in group} ES'_{j,t} + eps)   (Eq. 13-14)
    `esp_keys`: values the Eq. 12 top-K_e is taken over (default ES' in fp64;
    the float32 ES' of the spec mode when integer parity is wanted).
    """
    N_g, N, N_e = cfg.n_groups, cfg.experts_per_group, cfg.n_experts
    GS = np.asarray(GS, np.float64)
    ESp = np.asarray(ESp, np.float64)
    T = GS.shape[0]
    cG = np.bincount(np.asarray(group_idx).ravel(), minlength=N_g).astype(np.int64)
    sG = (GS / GS.sum(axis=1, keepdims=True)).sum(axis=0)
    cE_route = np.bincount(np.asarray(expert_idx).ravel(), minlength=N_e).astype(np.int64)
    gsel = np.zeros((T, N_g), bool)
    gsel[np.arange(T)[:, None], group_idx] = True
    keys = ESp if esp_keys is None else np.asarray(esp_keys)
    keys = np.where(np.repeat(gsel, N, axis=1), keys, -1.0)
    lit_idx = topk_rounds(keys, cfg.k_experts)
    cE_lit = np.bincount(lit_idx.ravel(), minlength=N_e).astype(np.int64)
    gsum = ESp.reshape(T, N_g, N).sum(axis=2, keepdims=True)
    sE = (ESp.reshape(T, N_g, N) / (gsum + cfg.eps)).sum(axis=0).reshape(N_e)
    out = dict(cG=cG, sG=sG, cE_route=cE_route, cE_lit=cE_lit, sE=sE, lit_idx=lit_idx)
    out.update(aux_losses(cfg, T, cG, sG, cE_lit if cfg.fe_mode == 0 else cE_route, sE))
    return out


def aux_losses(cfg: OracleConfig, T, cG, sG, cE, sE):
    """L_G (Eq. 7) and L_E (Eq. 11) from the raw statistics over T tokens."""
    N_g, N = cfg.n_groups, cfg.experts_per_group
    W = np.asarray(cfg.group_width, np.float64)
    fnorm = 1.0 / T if cfg.f_norm_by_T else 1.0
    fG = (N_g / cfg.k_groups) * np.asarray(cG, np.float64) * fnorm      # Eq. 8
    pG = np.asarray(sG, np.float64) / T                                 # Eq. 9
    fE = (N / cfg.k_experts) * np.asarray(cE, np.float64) * fnorm       # Eq. 12
    pE = np.asarray(sE, np.float64) / T                                 # Eq. 13
    L_G = cfg.alpha_g * float(np.sum(W / W.max() * fG * pG))            # Eq. 7
    L_E = cfg.alpha_e * float(np.sum(fE * pE))                          # Eq. 11
    return dict(fG=fG, pG=pG, fE=fE, pE=pE, L_G=L_G, L_E=L_E)


# --------------------------------------------------------------------------
# Token permutation (dispatch).  Not in the paper: the stable counting sort
# by expert, then token, that any grouped-expert execution needs.
# --------------------------------------------------------------------------

def dispatch(expert_idx, n_experts, row_align=1):
    """counts, offsets (exclusive prefix sum), row_of[t,k], src_of[row].

    Rows of expert e occupy [offsets[e], offsets[e+1]) in ascending (t, k)
    order.  `aligned_offsets` places every expert segment at a multiple of
    `row_align` physical rows; prow_of is row_of in that padded numbering."""
    expert_idx = np.asarray(expert_idx)
    T, K = expert_idx.shape
    counts = np.zeros(n_experts, np.int32)
    for e in expert_idx.ravel():
        counts[e] += 1
    offsets = np.zeros(n_experts + 1, np.int32)
    aligned = np.zeros(n_experts + 1, np.int32)
    for e in range(n_experts):
        offsets[e + 1] = offsets[e] + counts[e]
        padded = (counts[e] + row_align - 1) // row_align * row_align
        aligned[e + 1] = aligned[e] + padded
    fill = np.zeros(n_experts, np.int64)
    row_of = np.empty((T, K), np.int32)
    prow_of = np.empty((T, K), np.int32)
    src_of = np.empty(T * K, np.int32)
    for t in range(T):
        for k in range(K):
            e = expert_idx[t, k]
            row_of[t, k] = offsets[e] + fill[e]
            prow_of[t, k] = aligned[e] + fill[e]
            src_of[row_of[t, k]] = t * K + k
            fill[e] += 1
    return dict(counts=counts, offsets=offsets, aligned_offsets=aligned,
                row_of=row_of, prow_of=prow_of, src_of=src_of)


def permute_rows(x, prow_of, n_rows):
    """x_perm[prow_of[t,k], :] = x[t, :]; rows nobody maps to are zero."""
    x = np.asarray(x)
    out = np.zeros((n_rows, x.shape[1]), x.dtype)
    T, K = prow_of.shape
    for k in range(K):
        out[prow_of[:, k]] = x
    return out


# --------------------------------------------------------------------------
# Experts, combine, backward
# --------------------------------------------------------------------------

def _sigmoid(a):
    return 1.0 / (1.0 + np.exp(-a))


def swiglu_ffn(xe, w13_e, w2_e):
    """One expert of hidden width W: W_down( silu(W_gate x) * (W_up x) ).

    w13_e [2W, d]: rows 0..W-1 gate projection, rows W..2W-1 up projection.
    w2_e  [d, W]: down projection."""
    W = w2_e.shape[1]
    A = xe @ w13_e[:W].T
    U = xe @ w13_e[W:].T
    H = A * _sigmoid(A) * U
    return A, U, H, H @ w2_e.T


def _as64(a):
    return np.asarray(a, np.float64)


def expert_backward(xe, w13_e, w2_e, A, U, H, dY):
    """Gradients of one SwiGLU expert given dY = d<loss>/dY for its rows.

    With Y = H W_down^T, H = silu(A) * U, A = X W_gate^T, U = X W_up^T:
    dH = dY W_down; dW_down = dY^T H; dA = dH * U * silu'(A); dU = dH * silu(A);
    dW13 = [dA | dU]^T X; dX = dA W_gate + dU W_up."""
    W = w2_e.shape[1]
    dH = dY @ w2_e
    dw2 = dY.T @ H
    sg = _sigmoid(A)
    dA = dH * U * sg * (1.0 + A * (1.0 - sg))
    dU = dH * A * sg
    dw13 = np.concatenate([dA.T @ xe, dU.T @ xe], axis=0)
    dx = dA @ w13_e[:W] + dU @ w13_e[W:]
    return dict(dH=dH, dA=dA, dU=dU, dw2=dw2, dw13=dw13, dx=dx)


def layer_forward(cfg: OracleConfig, x, w_r, w13: List, w2: List, logit_bias=None,
                  logits=None, mode="definition", shared=None):
    """Forward of the whole layer.

    y_t = sum over the K_e selected experts of ES_{g,i,t} * E_{g,i}(x_t)
    (appendix Eq. 15 with the gate of Eq. 6).  mode "definition": selection in
    fp64 (Eq. 2-6).  mode "spec": the integer selection comes from the float32
    contract, all real values are still evaluated in fp64 for that selection.
    `shared` = (w13_s [2*W_s, d], w2_s [d, W_s]): the always-active shared experts of the
    paper's models (App. A.2 lists N_s = 2 of them without an equation).  Reading: as in the
    DeepSeek-V2 layer the baseline is adapted from, they are FFNs applied to every token and
    added to the routed sum with no gate; N_s such FFNs of width W equal one FFN of width
    N_s * W with the weights concatenated along the hidden axis, which is what is passed here.
    Returns a dict with every intermediate needed by tests and by the backward.
    """
    cfg.check()
    x = _as64(x)
    w_r = _as64(w_r)
    T, d = x.shape
    N = cfg.experts_per_group
    if logits is None:
        logits = router_logits(x, w_r, logit_bias)
    logits = _as64(logits)
    if mode == "definition":
        r = route_definition(cfg, logits)
        esp_keys = None
    elif mode == "spec":
        s = route_spec(cfg, logits.astype(np.float32))
        v = route_values(cfg, logits, s["group_idx"])
        r = dict(group_idx=s["group_idx"], expert_idx=s["expert_idx"],
                 gate=gates_from_selection(v["ESpp"], s["expert_idx"]), **v)
        esp_keys = s["ESp"]
    else:
        raise ValueError(mode)
    stats = aux_stats(cfg, r["GS"], r["ESp"], r["group_idx"], r["expert_idx"], esp_keys)
    y = np.zeros((T, d))
    per_expert = {}
    for e in range(cfg.n_experts):
        g, i = divmod(e, N)
        t_idx, k_idx = np.nonzero(r["expert_idx"] == e)        # ascending t
        if t_idx.size == 0:
            continue
        A, U, H, Y = swiglu_ffn(x[t_idx], _as64(w13[g][i]), _as64(w2[g][i]))
        np.add.at(y, t_idx, r["gate"][t_idx, k_idx][:, None] * Y)
        per_expert[e] = dict(t=t_idx, k=k_idx, A=A, U=U, H=H, Y=Y)
    shared_saved = None
    if shared is not None:
        A, U, H, Y = swiglu_ffn(x, _as64(shared[0]), _as64(shared[1]))
        y = y + Y
        shared_saved = dict(A=A, U=U, H=H, Y=Y)
    return dict(cfg=cfg, x=x, w_r=w_r, logits=logits, y=y, per_expert=per_expert,
                stats=stats, shared=shared_saved, **r)


def layer_loss(fwd, G):
    """Scalar used by the gradient checks: <y, G> + L_G + L_E."""
    return float(np.sum(fwd["y"] * _as64(G))) + fwd["stats"]["L_G"] + fwd["stats"]["L_E"]


def layer_backward(fwd, w13: List, w2: List, dy, with_aux=True, aux_counts=None, shared=None):
    """Gradients of  <y, dy> (+ L_G + L_E when with_aux)  w.r.t. x, the router
    weight and every expert weight.  Top-k choices and the indicator counts
    f^G, f^E are piecewise constant and carry no gradient.

    aux_counts = (cG, cE, T_total) overrides the statistics of this batch (used
    when `fwd` holds only a sample of the tokens of a larger batch)."""
    cfg: OracleConfig = fwd["cfg"]
    N_g, N, N_e = cfg.n_groups, cfg.experts_per_group, cfg.n_experts
    x, w_r = fwd["x"], fwd["w_r"]
    dy = _as64(dy)
    T, d = x.shape
    gate, expert_idx = fwd["gate"], fwd["expert_idx"]
    dx = np.zeros_like(x)
    dgate = np.zeros_like(gate)
    dw13 = [np.zeros(np.shape(w), np.float64) for w in w13]
    dw2 = [np.zeros(np.shape(w), np.float64) for w in w2]
    for e, c in fwd["per_expert"].items():
        g, i = divmod(e, N)
        W = cfg.group_width[g]
        t_idx, k_idx, A, U, H, Y = c["t"], c["k"], c["A"], c["U"], c["H"], c["Y"]
        w13_e, w2_e = _as64(w13[g][i]), _as64(w2[g][i])
        dgate[t_idx, k_idx] = np.sum(dy[t_idx] * Y, axis=1)
        dY = gate[t_idx, k_idx][:, None] * dy[t_idx]
        eb = expert_backward(x[t_idx], w13_e, w2_e, A, U, H, dY)
        dw2[g][i] = eb["dw2"]
        dw13[g][i] = eb["dw13"]
        np.add.at(dx, t_idx, eb["dx"])
    # ---- router: Eq. 6 -> Eq. 4 -> Eq. 3 -> Eq. 2 ----
    GS, ESp, ESpp = fwd["GS"], fwd["ESp"], fwd["ESpp"]
    key = np.take_along_axis(ESpp, expert_idx.astype(np.int64), axis=1)
    ssum = key.sum(axis=1, keepdims=True)
    dkey = (dgate - np.sum(dgate * gate, axis=1, keepdims=True)) / ssum
    dESpp = np.zeros((T, N_e))
    np.put_along_axis(dESpp, expert_idx.astype(np.int64), dkey, axis=1)
    ESp3 = ESp.reshape(T, N_g, N)
    dESpp3 = dESpp.reshape(T, N_g, N)
    dGS = np.sum(dESpp3 * ESp3, axis=2)
    dESp3 = dESpp3 * GS[:, :, None]
    if with_aux:
        if aux_counts is None:
            st = fwd["stats"]
            cG, cE, Ttot = st["cG"], (st["cE_lit"] if cfg.fe_mode == 0 else st["cE_route"]), T
        else:
            cG, cE, Ttot = aux_counts
        fnorm = 1.0 / Ttot if cfg.f_norm_by_T else 1.0
        Wd = np.asarray(cfg.group_width, np.float64)
        cg = Wd / Wd.max() * (N_g / cfg.k_groups) * _as64(cG) * fnorm
        fE = ((N / cfg.k_experts) * _as64(cE) * fnorm).reshape(1, N_g, N)
        Ssum = GS.sum(axis=1, keepdims=True)
        dGS = dGS + cfg.alpha_g / Ttot * (cg[None, :] / Ssum
                                          - np.sum(cg[None, :] * GS, axis=1, keepdims=True) / Ssum ** 2)
        D = ESp3.sum(axis=2, keepdims=True) + cfg.eps
        dS = cfg.alpha_e / Ttot * (fE / D - np.sum(fE * ESp3, axis=2, keepdims=True) / D ** 2)
        dESp3 = dESp3 + np.where(fwd["group_mask"][:, :, None], dS, 0.0)
    dlE = ESp3 * (dESp3 - np.sum(ESp3 * dESp3, axis=2, keepdims=True))
    dlG = dGS * GS * (1.0 - GS)
    dlogits = np.concatenate([dlG, dlE.reshape(T, N_e)], axis=1)
    dw_r = dlogits.T @ x
    dx_router = dlogits @ w_r
    out = dict(dx_experts=dx, dx_router=dx_router, dw_r=dw_r, dw13=dw13, dw2=dw2, dgate=dgate,
               dlogits=dlogits)
    dx_total = dx + dx_router
    if shared is not None:
        # the shared FFN sees every token with unit gate: dY = dy
        c = fwd["shared"]
        sb = expert_backward(x, _as64(shared[0]), _as64(shared[1]), c["A"], c["U"], c["H"], dy)
        dx_total = dx_total + sb["dx"]
        out.update(shared=sb)
    out["dx"] = dx_total
    return out
