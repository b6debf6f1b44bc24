"""The allocation-free statistics entry point against the workspace-based one.

Some callers cannot give the library a workspace because they cannot allocate at that point
(device memory fully owned by a framework pool, or a loop that must avoid cudaMalloc's implicit
synchronisation).  `mohge_aux_stats_static` serves them from a scratch array built into the
library.  It must return exactly what `mohge_aux_stats` returns, on repeated calls (the array
keeps the previous call's contents), and refuse configs beyond its stated limit.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from paper_2604_23108_b200 import binding as B
from paper_2604_23108_b200.inputs import Workload, make_inputs

pytestmark = pytest.mark.gpu


def _routed(wl, seed):
    cfg = B.Config(d_model=wl.d_model, n_groups=wl.n_groups, experts_per_group=wl.experts_per_group,
                   k_groups=wl.k_groups, k_experts=wl.k_experts, group_width=list(wl.group_width),
                   dtype=wl.dtype, row_align=1)
    inp = make_inputs(wl, seed=seed, weights=False)
    b = B.LayerBuffers(cfg, wl.T)
    B.mohge_route(cfg, wl.T, inp["x"].cuda(), inp["w_router"].cuda(), None, None, b.logits,
                  b.group_idx, b.expert_idx, b.gate_w, b.gs, b.esp, b.ws)
    return cfg, b


def _stats_outputs(cfg, dev):
    i32, f32 = torch.int32, torch.float32
    return dict(gc=torch.empty(cfg.n_groups, dtype=i32, device=dev),
                gp=torch.empty(cfg.n_groups, dtype=f32, device=dev),
                cr=torch.empty(cfg.n_experts, dtype=i32, device=dev),
                cl=torch.empty(cfg.n_experts, dtype=i32, device=dev),
                ep=torch.empty(cfg.n_experts, dtype=f32, device=dev),
                loss=torch.empty(4, dtype=f32, device=dev))


def test_static_scratch_matches_workspace_version_twice_in_a_row():
    # Different batches back to back: every call meets the previous call's leftovers.  The third
    # repeats the first workload after the smaller one, so a batch with few partial rows is
    # followed by one that has to overwrite every stale row.  Both entry points run the same
    # kernels with the same fixed-order sums, so even the float results must agree bit for bit.
    big, small = Workload("na1", "f32", 3000, 64, 4, 16, (32, 24, 16, 8), 2, 6), Workload("na2", "f32", 777, 64, 3, 5, (32, 24, 16), 2, 4)
    for wl, seed in ((big, 21), (small, 22), (big, 23)):
        cfg, b = _routed(wl, seed)
        ref, got = _stats_outputs(cfg, "cuda"), _stats_outputs(cfg, "cuda")
        B.mohge_aux_stats(cfg, wl.T, b.gs, b.esp, b.group_idx, b.expert_idx, ref["gc"], ref["gp"],
                          ref["cr"], ref["cl"], ref["ep"], ref["loss"], b.ws)
        B.mohge_aux_stats_static(cfg, wl.T, b.gs, b.esp, b.group_idx, b.expert_idx, got["gc"],
                                 got["gp"], got["cr"], got["cl"], got["ep"], got["loss"])
        torch.cuda.synchronize()
        for k in ("gc", "cr", "cl"):
            assert torch.equal(ref[k], got[k]), k                        # integer counts: exact
        assert int(got["gc"].sum()) == wl.T * wl.k_groups
        for k in ("gp", "ep"):
            assert torch.equal(ref[k], got[k]), k                        # same bits, not just close
        assert torch.equal(ref["loss"][:2], got["loss"][:2])


def test_static_scratch_refuses_configs_beyond_its_limit():
    cfg = B.Config(d_model=64, n_groups=8, experts_per_group=32, k_groups=3, k_experts=6,
                   group_width=[8] * 8, dtype="f32", row_align=1)       # 8 + 256 outputs > 136
    one = C.c_void_p(256)
    rc = B.lib().mohge_aux_stats_static(C.byref(cfg.c()), 16, *([one] * 10), None)
    assert rc == -1
    msg = B.lib().mohge_last_error().decode()
    assert "136" in msg and "mohge_aux_stats" in msg
