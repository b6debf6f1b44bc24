"""Helpers shared by the GPU parity tests: config conversion, oracle runs, error metrics."""
from __future__ import annotations

import numpy as np
import torch

import oracle as O
from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import Workload, make_inputs


def to_np64(t: torch.Tensor) -> np.ndarray:
    return t.detach().to("cpu").to(torch.float64).numpy()


def oracle_cfg(wl: Workload, **kw) -> O.OracleConfig:
    return O.OracleConfig(d_model=wl.d_model, n_groups=wl.n_groups,
                          experts_per_group=wl.experts_per_group, k_groups=wl.k_groups,
                          k_experts=wl.k_experts, group_width=list(wl.group_width), **kw)


def gpu_cfg(wl: Workload, **kw) -> B.Config:
    kw.setdefault("row_align", 128 if wl.dtype == "bf16" else 1)
    return B.Config(d_model=wl.d_model, n_groups=wl.n_groups,
                    experts_per_group=wl.experts_per_group, k_groups=wl.k_groups,
                    k_experts=wl.k_experts, group_width=list(wl.group_width), dtype=wl.dtype, **kw)


def max_rel(a, b) -> float:
    """max|a - b| / max|b| (the tolerance metric of the parity bar)."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    den = np.max(np.abs(b))
    if den == 0:
        return float(np.max(np.abs(a)))
    return float(np.max(np.abs(a - b)) / den)


def elementwise_outliers(a, b, tol) -> float:
    """Share of elements with |a - b| > tol |b| + tol rms(b): the secondary, element-wise figure
    reported beside max_rel (a per-tensor maximum cannot see a large relative error on a small
    element; this one can, down to elements of the size of tol rms)."""
    a = np.asarray(a, np.float64)
    b = np.asarray(b, np.float64)
    if b.size == 0:
        return 0.0
    rms = float(np.sqrt(np.mean(b * b)))
    return float(np.mean(np.abs(a - b) > tol * np.abs(b) + tol * rms))


def tol_for(dtype: str) -> float:
    return 2e-2 if dtype == "bf16" else 1e-5


def oracle_layer(wl: Workload, inp, ocfg=None, with_aux=True, logits32=None):
    """Oracle forward + backward.  Routing takes the float32 logits `logits32`
    (default: the oracle's own fp64 logits rounded to float32) in spec mode."""
    ocfg = ocfg or oracle_cfg(wl)
    x, w_r = to_np64(inp["x"]), to_np64(inp["w_router"])
    w13 = [to_np64(w) for w in inp["w13"]]
    w2 = [to_np64(w) for w in inp["w2"]]
    bias = None if inp.get("logit_bias") is None else to_np64(inp["logit_bias"])
    if logits32 is None:
        logits32 = O.router_logits(x, w_r, bias).astype(np.float32)
    fwd = O.layer_forward(ocfg, x, w_r, w13, w2, logits=logits32.astype(np.float64), mode="spec")
    bwd = O.layer_backward(fwd, w13, w2, to_np64(inp["dy"]), with_aux=with_aux)
    return fwd, bwd, logits32


def gpu_layer(wl: Workload, inp, gcfg=None, logits32=None, with_aux=True, accumulate=False):
    """Full forward + backward through the C ABI; returns (buffers, device inputs)."""
    gcfg = gcfg or gpu_cfg(wl)
    T = inp["x"].shape[0]
    dev = {k: (v.cuda() if isinstance(v, torch.Tensor) else v) for k, v in inp.items()
           if k not in ("w13", "w2")}
    dev["w13"] = [w.cuda() for w in inp["w13"]]
    dev["w2"] = [w.cuda() for w in inp["w2"]]
    b = B.LayerBuffers(gcfg, T)
    lg = None if logits32 is None else torch.from_numpy(np.ascontiguousarray(logits32)).cuda()
    B.layer_forward(gcfg, b, dev["x"], dev["w_router"], dev["w13"], dev["w2"],
                    logit_bias=dev.get("logit_bias"), logits_in=lg, aux=True)
    B.layer_backward(gcfg, b, dev["x"], dev["w_router"], dev["w13"], dev["w2"], dev["dy"],
                     aux=with_aux, accumulate=accumulate)
    torch.cuda.synchronize()
    assert B.mohge_get_device_status(b.ws) == 0
    return b, dev


class forced_switches:
    """Context manager: sets debugging switches of the library ("MOHGE_TC_CG=2,MOHGE_TC_WIDE=63"
    in the spelling of their environment variables) and puts the library's own rules back after."""

    def __init__(self, spec: str):
        self.items = [kv.split("=") for kv in spec.split(",") if kv]

    @staticmethod
    def _name(env_name: str) -> str:
        return env_name[len("MOHGE_"):].lower()

    def __enter__(self):
        for name, value in self.items:
            B.mohge_set_switch(self._name(name), int(value))
        return self

    def __exit__(self, *exc):
        for name, _ in self.items:
            B.mohge_set_switch(self._name(name), -1)
        return False
