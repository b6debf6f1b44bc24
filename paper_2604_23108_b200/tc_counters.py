"""Per-CTA clock counters of the grouped GEMM kernel, per role, over a few layer steps.

    python -m paper_2604_23108_b200.build --counters
    python -m paper_2604_23108_b200.tc_counters --workload cfg4_bf16_skew [--steps 20]

Runs forward + backward of the layer with libmohge_counters.so (the library compiled with
-DMOHGE_TC_COUNTERS) and prints, for every role of tc_grouped_kernel:
  * the time of a launch (longest CTA lifetime) and the achieved TFLOP/s,
  * the balance of the tile scheduler: shortest and longest CTA busy time over the mean,
  * clocks per k-block (one 256 x 256 x 64 block of MMAs; 512 = tensor-pipe peak) over the whole
    launch and in the middle of long tiles (steady state),
  * the share of the MMA issuer's time spent waiting for an accumulator (exposed epilogue) and for
    operands (loads not keeping up), and the share of the epilogue warps' time spent waiting for MMAs.
MOHGE_TC_WIDE=<mask>, MOHGE_TC_CG=1|2 and MOHGE_TC_GRID=<n> select tile forms and the number of CTAs.
"""
from __future__ import annotations

import argparse
import ctypes as C
import os

import numpy as np
import torch

from . import binding as B
from .inputs import WORKLOADS, make_device_inputs

ROLES = ["FWD1", "FWD2", "DGRAD_DOWN", "DGRAD_13", "WGRAD_DOWN", "WGRAD_13", "LOGITS", "ROUTER_DW", "ROUTER_DX"]
FLOP_SHARE = {0: 4, 1: 2, 2: 2, 3: 4, 4: 2, 5: 4}     # of the 18 d W FLOPs per routed row


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg5_slice", choices=list(WORKLOADS))
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--gather", action="store_true",
                    help="use the entry points that gather the rows of x instead of reading x_perm")
    args = ap.parse_args()
    B.LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libmohge_counters.so")
    wl = WORKLOADS[args.workload]
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    cfg = B.Config(d_model=wl.d_model, n_groups=wl.n_groups, experts_per_group=wl.experts_per_group,
                   k_groups=wl.k_groups, k_experts=wl.k_experts, group_width=list(wl.group_width),
                   dtype=wl.dtype)
    inp = make_device_inputs(wl, dev)
    b = B.LayerBuffers(cfg, wl.T, device=dev)
    lib = B.lib()
    lib.mohge_debug_tc_counters.restype = C.c_int32
    lib.mohge_debug_tc_counters.argtypes = [C.c_void_p, C.c_int32]
    cnt = np.zeros((9, 160, 12), dtype=np.uint64)

    def step():
        B.layer_forward(cfg, b, inp["x"], inp["w_router"], inp["w13"], inp["w2"],
                        logit_bias=inp["logit_bias"], aux=True, gather=args.gather)
        B.layer_backward(cfg, b, inp["x"], inp["w_router"], inp["w13"], inp["w2"], inp["dy"], aux=True,
                         gather=args.gather)

    for _ in range(args.warmup):
        step()
    assert lib.mohge_debug_tc_counters(cnt.ctypes.data, 1) == 0
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / args.steps
    assert lib.mohge_debug_tc_counters(cnt.ctypes.data, 1) == 0
    assert B.mohge_get_device_status(b.ws) == 0
    counts = b.counts.cpu().numpy()
    N = wl.experts_per_group
    rows_w = sum(float(m) * wl.group_width[e // N] for e, m in enumerate(counts))
    cmax, cmin = counts.max(), counts[counts > 0].min()
    print("workload %s%s: %.3f ms per step, %.0f tokens/s; tokens per expert min %d max %d (x%.0f)"
          % (wl.name, " (gathering entry points)" if args.gather else "", ms, wl.T / ms * 1e3, cmin, cmax, cmax / cmin))
    print("| role | CTAs | ms per launch | TFLOP/s | busy min/mean | busy max/mean | clocks per k-block | steady state "
          "| issuer waits for accumulator | issuer waits for operands | epilogue warps wait for MMAs |")
    print("|---|---|---|---|---|---|---|---|---|---|---|")
    total_ms = 0.0
    for r in range(9):
        c = cnt[r].astype(np.float64)
        act = c[:, 7] > 0
        if not act.any():
            continue
        life = c[act, 7]
        kern_ms = life.max() / args.steps / 1e6
        lead = c[:, 1] > 0                              # CTAs that issue MMAs (pair leaders)
        busy = c[lead, 1]
        tf = ""
        if r in FLOP_SHARE:
            tf = "%.0f" % (FLOP_SHARE[r] * wl.d_model * rows_w / (kern_ms * 1e-3) / 1e12)
            total_ms += kern_ms
        kb = c[lead, 9].sum()
        steady = "%.0f" % (c[lead, 10].sum() / c[lead, 11].sum()) if c[lead, 11].sum() > 0 else ""
        epi = c[act, 6].sum()
        print("| %s | %d | %.3f | %s | %.3f | %.3f | %.0f | %s | %.1f %% | %.1f %% | %.1f %% |"
              % (ROLES[r], int(act.sum()), kern_ms, tf, busy.min() / busy.mean(), busy.max() / busy.mean(),
                 busy.sum() / kb if kb else 0.0, steady, 100.0 * c[lead, 3].sum() / busy.sum(),
                 100.0 * c[lead, 2].sum() / busy.sum(), 100.0 * c[act, 5].sum() / epi if epi else 0.0))
    print("six expert GEMMs: %.3f ms per step = %.0f TFLOP/s" % (total_ms, 18.0 * wl.d_model * rows_w / (total_ms * 1e-3) / 1e12))


if __name__ == "__main__":
    main()
