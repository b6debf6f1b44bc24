#!/usr/bin/env python
"""Benchmark of the MoHGE expert layer forward + backward on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one pass of the whole hot path over one batch: route (logits GEMM + two-level
selection), auxiliary statistics, dispatch, grouped SwiGLU experts forward, combine, and the full
backward (combine, experts dgrad + wgrad, dispatch, router).  The metric is tokens/s of that
step.  With N > 1 every rank runs an independent replica of the layer (the path does not shard:
"replicas only"), timed as the maximum over ranks.

`--impl reference` times the fp64 numpy oracle on the host cores on a bounded sample of the
same workload (there is no reference implementation of this layer to run).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2604_23108_b200.inputs import WORKLOADS, Workload, make_device_inputs  # noqa: E402

# DRAM bytes (read + written) of the six grouped-GEMM launches of one step, from a counter capture
# of the kernels as they stand now.  The large workload is too big to capture with counters; its
# figure is the capture of "cfg5_slice" (one eighth of the experts, the same tokens per expert,
# widths and tile forms) times eight: every expert's tiles are independent problems, so the traffic
# grows with the number of experts.  None: no capture of the current kernels.
NCU_DRAM_TRAFFIC_PER_STEP = {"cfg5_bf16_large": 8 * 8.825e9, "cfg5_slice": 8.825e9}
NCU_DRAM_TRAFFIC_SOURCE = {
    "cfg5_bf16_large": "ncu counters of the six launches at cfg5_slice (one eighth of the experts, same tokens per "
                       "expert, widths and tile forms) times 8; not measured in this run",
    "cfg5_slice": "ncu counters of the six launches of one step; not measured in this run",
}

METRIC = "MoHGE layer fwd+bwd tokens/s"
METRIC_FWD = "MoHGE layer fwd tokens/s"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "cfg5_bf16_large"


def _peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return dict(hbm=d["hbm_gbs"], tf_burst=d["bf16_tflops"], tf_sustained=d["bf16_tflops_sustained"],
                    source="measured")
    return dict(hbm=6650.0, tf_burst=1590.0, tf_sustained=1400.0, source="fallback")


class ClockSampler:
    """nvidia-smi clocks and throttle reasons sampled every 200 ms while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(gpu_index), "--query-gpu=" + self.Q,
                                       "--format=csv,noheader,nounits", "-lms", "200"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = dict(sm_mhz=None, sm_max_mhz=None, reasons=[], samples=0)
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, smax, pw, reasons = [], [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            c = [v.strip() for v in line.split(",")]
            if len(c) < 9:
                continue
            try:
                sm.append(float(c[1]))
                smax.append(float(c[2]))
                pw.append(float(c[3]))
            except ValueError:
                continue
            for n, v in zip(names, c[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), samples=len(sm),
                       power_w=statistics.median(pw))
        out["reasons"] = sorted(reasons)
        return out


ORACLE_SAMPLE_TOKENS = 256      # the one sample size of both oracle arms (cpu_baseline and --impl reference)
ORACLE_BUDGET_S = 120.0         # timed oracle steps stop once this much time has been spent


def oracle_sample_run(wl: Workload, sample_tokens: int, steps: int, warmup: int, inp_cpu=None,
                      budget_s: float = ORACLE_BUDGET_S):
    """Times the oracle (as it stands) on `sample_tokens` tokens of the workload.  Returns
    (tokens/s, seconds per step, steps run, seconds to convert every expert's weights to fp64).
    The oracle's step time is dominated by that conversion, which it repeats for every expert a
    step touches, so tokens/s is not linear in the sample: both oracle arms use the same sample."""
    import numpy as np
    import oracle as O
    from paper_2604_23108_b200.inputs import make_inputs
    if inp_cpu is None:
        inp_cpu = make_inputs(wl, T=sample_tokens)
    to_np64 = lambda t: t.detach().to("cpu").to(torch.float64).numpy()
    ocfg = O.OracleConfig(d_model=wl.d_model, n_groups=wl.n_groups, experts_per_group=wl.experts_per_group,
                          k_groups=wl.k_groups, k_experts=wl.k_experts, group_width=list(wl.group_width))
    x, w_r, dy = to_np64(inp_cpu["x"][:sample_tokens]), to_np64(inp_cpu["w_router"]), to_np64(inp_cpu["dy"][:sample_tokens])
    bias = None if inp_cpu.get("logit_bias") is None else to_np64(inp_cpu["logit_bias"])
    w13, w2 = inp_cpu["w13"], inp_cpu["w2"]       # converted to fp64 expert by expert inside the oracle
    w13n = [w.to(torch.float32).numpy() for w in w13]
    w2n = [w.to(torch.float32).numpy() for w in w2]
    t0 = time.perf_counter()
    for w in w13n + w2n:
        w.astype(np.float64)
    t_conv = time.perf_counter() - t0
    times, spent = [], 0.0
    for it in range(warmup + steps):
        t0 = time.perf_counter()
        fwd = O.layer_forward(ocfg, x, w_r, w13n, w2n, logit_bias=bias, mode="spec")
        O.layer_backward(fwd, w13n, w2n, dy, with_aux=True)
        t1 = time.perf_counter()
        spent += t1 - t0
        if it >= warmup:
            times.append(t1 - t0)
            if spent > budget_s:
                break
    per = sum(times) / len(times)
    return sample_tokens / per, per, len(times), t_conv


def oracle_baseline_dict(val, per, n, t_conv, sample, cores):
    return {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "steps_run": n,
            "sample": "oracle fwd+bwd on the first %d tokens of the workload, all experts' weights "
                      "(%.1f s per step, of which about %.1f s convert the weights of the experts hit to "
                      "fp64)" % (sample, per, min(per, 2.0 * t_conv))}


def run_reference(args, wl: Workload, rank: int):
    if rank != 0:
        return
    from paper_2604_23108_b200.inputs import make_inputs
    cores = torch.get_num_threads()
    sample = min(wl.T, ORACLE_SAMPLE_TOKENS)
    inp_cpu = make_inputs(wl, T=sample)
    # the same sample as the cpu_baseline leg of the default line; as many of the requested steps
    # as fit into the time budget (one warm-up step at most)
    val, per, n, t_conv = oracle_sample_run(wl, sample, max(1, args.steps), min(args.warmup, 1), inp_cpu=inp_cpu)
    line = {
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
        "data": "synthetic",
        "config": {"workload": wl.name, "T": wl.T, "d_model": wl.d_model,
                   "sample": "first %d tokens, all experts" % sample, "steps_run": n},
        "cpu_baseline": oracle_baseline_dict(val, per, n, t_conv, sample, cores),
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line), flush=True)


def max_over_ranks(ms: float, dist, device) -> float:
    """Slowest rank's time: the number a multi-replica run is judged by (dist None: one rank)."""
    if dist is None:
        return ms
    t = torch.tensor([ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def replica_seed(wl: Workload, rank: int) -> int:
    """Every rank runs an independent replica of the layer on its own seeded batch."""
    return wl.seed + rank


def flops_per_step(wl: Workload, counts, shared_width: int = 0) -> float:
    """Algorithmic FLOPs of the expert GEMMs: 18 * d * sum_e M_e * W_g(e) (fwd 6, bwd 12), plus
    18 * d * T * shared_width when shared experts run."""
    N = wl.experts_per_group
    tot = float(wl.T) * shared_width
    for e, m in enumerate(counts):
        tot += float(m) * wl.group_width[e // N]
    return 18.0 * wl.d_model * tot


def make_step(B, gcfg, T, inp, buf, shared=None, shared_width=0, forward_only=False, gather=False,
              dy_fused=False):
    """One pass of the whole hot path through the C ABI.  Returns (step, gemm_marks): with
    mark=True a step records CUDA events around mohge_expert_fwd and mohge_expert_bwd_dgate."""
    ev = lambda: torch.cuda.Event(enable_timing=True)
    gemm_marks = []

    def step(mark=False, y=None, dx=None, after_fwd=None, before_bwd=None):
        y = buf.y if y is None else y
        dx = buf.dx if dx is None else dx
        B.mohge_route(gcfg, T, inp["x"], inp["w_router"], inp["logit_bias"], None, buf.logits,
                      buf.group_idx, buf.expert_idx, buf.gate_w, buf.gs, buf.esp, buf.ws)
        B.mohge_aux_stats(gcfg, T, buf.gs, buf.esp, buf.group_idx, buf.expert_idx, buf.group_count,
                          buf.group_psum, buf.cnt_routed, buf.cnt_lit, buf.expert_psum, buf.loss, buf.ws)
        if gather:      # no x_perm: the GEMMs gather the rows of x
            B.mohge_dispatch_indices(gcfg, T, buf.expert_idx, buf.counts, buf.offsets, buf.aligned,
                                     buf.row_of, buf.prow_of, buf.src_of, buf.tok_of_prow, buf.ws)
        else:
            B.mohge_dispatch(gcfg, T, inp["x"], buf.expert_idx, buf.counts, buf.offsets, buf.aligned,
                             buf.row_of, buf.prow_of, buf.src_of, buf.x_perm, buf.ws)
        if mark:
            e0, e1, e2, e3 = ev(), ev(), ev(), ev()
            e0.record()
        if gather:
            B.mohge_expert_fwd_gather(gcfg, T, inp["x"], buf.tok_of_prow, buf.counts, buf.aligned, inp["w13"],
                                      inp["w2"], buf.au, buf.h, buf.y_perm, buf.ws)
        else:
            B.mohge_expert_fwd(gcfg, T, buf.x_perm, buf.counts, buf.aligned, inp["w13"], inp["w2"],
                               buf.au, buf.h, buf.y_perm, buf.ws)
        if shared is not None:
            B.mohge_shared_fwd(gcfg, T, shared_width, inp["x"], shared[0], shared[1], buf.au_sh,
                               buf.h_sh, buf.y_sh, buf.ws)
        if mark:
            e1.record()
        B.mohge_combine(gcfg, T, buf.y_perm, buf.prow_of, buf.gate_w, y,
                        y_add=buf.y_sh if shared is not None else None)
        if after_fwd is not None:
            after_fwd()                     # y is final here (the end-to-end arm starts its download)
        if forward_only:
            if mark:
                gemm_marks.append((e0, e1, e1, e1))
            return
        if before_bwd is not None:
            before_bwd()                    # dy is first read below (the end-to-end arm waits for its upload)
        # the gate gradient comes out of the experts' backward, so combine_bwd reads no y_perm
        if dy_fused:    # no dy_perm: the GEMMs gather the rows of dy
            B.mohge_row_tokens(gcfg, T, buf.counts, buf.offsets, buf.aligned, buf.src_of, buf.tok_of_prow)
        else:
            B.mohge_combine_bwd(gcfg, T, inp["dy"], None, buf.prow_of, buf.gate_w, buf.counts,
                                buf.aligned, buf.dy_perm, None)
        if mark:
            e2.record()
        if dy_fused:
            B.mohge_expert_bwd_dy(gcfg, T, inp["dy"], buf.tok_of_prow, buf.x_perm, buf.au, buf.h, buf.counts,
                                  buf.aligned, inp["w13"], inp["w2"], buf.dau, buf.dx_perm, buf.dw13, buf.dw2,
                                  0, buf.y_perm, buf.prow_of, buf.gate_w, buf.dgate, buf.hs, buf.row_gate,
                                  buf.ws)
        elif gather:
            B.mohge_expert_bwd_gather(gcfg, T, buf.dy_perm, inp["x"], buf.tok_of_prow, buf.au, buf.h, buf.counts,
                                      buf.aligned, inp["w13"], inp["w2"], buf.dau, buf.dx_perm, buf.dw13,
                                      buf.dw2, 0, inp["dy"], buf.y_perm, buf.prow_of, buf.gate_w, buf.dgate,
                                      buf.ws)
        else:
            B.mohge_expert_bwd_dgate(gcfg, T, buf.dy_perm, buf.x_perm, buf.au, buf.h, buf.counts,
                                     buf.aligned, inp["w13"], inp["w2"], buf.dau, buf.dx_perm, buf.dw13,
                                     buf.dw2, 0, inp["dy"], buf.y_perm, buf.prow_of, buf.gate_w, buf.dgate,
                                     buf.ws)
        if shared is not None:
            B.mohge_shared_bwd(gcfg, T, shared_width, inp["dy"], inp["x"], buf.au_sh, buf.h_sh,
                               shared[0], shared[1], buf.dau_sh, buf.dx_sh, buf.dw13_sh, buf.dw2_sh,
                               0, buf.ws)
        if mark:
            e3.record()
            gemm_marks.append((e0, e1, e2, e3))
        B.mohge_dispatch_bwd(gcfg, T, buf.dx_perm, buf.prow_of, dx,
                             dx_add=buf.dx_sh if shared is not None else None)
        cnt_e = buf.cnt_lit if gcfg.fe_mode == 0 else buf.cnt_routed
        B.mohge_route_bwd(gcfg, T, inp["x"], inp["w_router"], buf.dgate, buf.gs, buf.esp,
                          buf.group_idx, buf.expert_idx, buf.group_count, cnt_e, buf.dlogits,
                          dx, buf.dw_router, buf.ws)

    return step, gemm_marks


def hbm_step_rooflines(B, gcfg, wl: Workload, inp, buf, hbm_peak_gbs: float, reps: int = 10):
    """CUDA-event time of every HBM-bound entry point of the step, each called `reps` times back
    to back on the buffers a full step has left behind, against its algorithmic bytes
    (s = bytes per element, R = T K_e routed rows, NL = N_g + N_e router outputs):
      route         x and the router weight read once, logits, scores, indices and gates
                    written: T d s + NL d s + 2 T NL 4 + T (8 K_e + 4 K_g)
      aux_stats     saved scores and indices read: T NL 4 + T (K_e + K_g) 4
      dispatch      (T + R) d s + 16 R (index arrays)
      combine       (R + T) d s          combine_bwd (scaled rows)  (T + R) d s
      dispatch_bwd  (R + T) d s          route_bwd   x read, dx read and written: 3 T d s + 2 T NL 4
    Small workloads fit in L2, where the figure exceeds the HBM rate; that is said in `l2`."""
    T, d, Ke, Kg, NL = wl.T, wl.d_model, wl.k_experts, wl.k_groups, wl.n_logits
    s_ = 2 if wl.dtype == "bf16" else 4
    R = T * Ke
    cnt_e = buf.cnt_lit if gcfg.fe_mode == 0 else buf.cnt_routed
    calls = {
        "route": (lambda: B.mohge_route(gcfg, T, inp["x"], inp["w_router"], inp["logit_bias"], None, buf.logits,
                                        buf.group_idx, buf.expert_idx, buf.gate_w, buf.gs, buf.esp, buf.ws),
                  T * d * s_ + NL * d * s_ + 2 * T * NL * 4 + T * (8 * Ke + 4 * Kg)),
        "aux_stats": (lambda: B.mohge_aux_stats(gcfg, T, buf.gs, buf.esp, buf.group_idx, buf.expert_idx,
                                                buf.group_count, buf.group_psum, buf.cnt_routed, buf.cnt_lit,
                                                buf.expert_psum, buf.loss, buf.ws),
                      T * NL * 4 + T * (Ke + Kg) * 4),
        "dispatch": (lambda: B.mohge_dispatch(gcfg, T, inp["x"], buf.expert_idx, buf.counts, buf.offsets,
                                              buf.aligned, buf.row_of, buf.prow_of, buf.src_of, buf.x_perm, buf.ws),
                     (T + R) * d * s_ + 16 * R),
        "combine": (lambda: B.mohge_combine(gcfg, T, buf.y_perm, buf.prow_of, buf.gate_w, buf.y),
                    (R + T) * d * s_),
        "combine_bwd": (lambda: B.mohge_combine_bwd(gcfg, T, inp["dy"], None, buf.prow_of, buf.gate_w, buf.counts,
                                                    buf.aligned, buf.dy_perm, None),
                        (T + R) * d * s_),
        "dispatch_bwd": (lambda: B.mohge_dispatch_bwd(gcfg, T, buf.dx_perm, buf.prow_of, buf.dx),
                         (R + T) * d * s_),
        "route_bwd": (lambda: B.mohge_route_bwd(gcfg, T, inp["x"], inp["w_router"], buf.dgate, buf.gs, buf.esp,
                                                buf.group_idx, buf.expert_idx, buf.group_count, cnt_e,
                                                buf.dlogits, buf.dx, buf.dw_router, buf.ws),
                      3 * T * d * s_ + 2 * T * NL * 4),
    }
    out = []
    for name, (fn, nbytes) in calls.items():
        fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / reps
        gbs = nbytes / (ms * 1e-3) / 1e9
        out.append({"step": name, "bound": "hbm", "bytes": nbytes, "ms": ms, "achieved": gbs,
                    "peak": hbm_peak_gbs, "unit": "GB/s", "frac": gbs / hbm_peak_gbs})
    return out


def count_ratio(counts):
    """Largest over smallest per-expert token count of the batch (None when an expert is empty)."""
    lo = min(counts)
    return None if lo == 0 else max(counts) / lo


def quick_workload_line(B, name: str, dev, pk, steps: int = 20, warmup: int = 3):
    """A short measurement of another benchmark workload for the default line's
    `other_workloads` list: tokens/s of the step and the rate of its grouped GEMMs."""
    wl = WORKLOADS[name]
    gcfg = B.Config(d_model=wl.d_model, n_groups=wl.n_groups, experts_per_group=wl.experts_per_group,
                    k_groups=wl.k_groups, k_experts=wl.k_experts, group_width=list(wl.group_width),
                    dtype=wl.dtype, row_align=128 if wl.dtype == "bf16" else 1)
    inp = make_device_inputs(wl, dev)
    buf = B.LayerBuffers(gcfg, wl.T, device=dev)
    step, marks = make_step(B, gcfg, wl.T, inp, buf)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t0 = time.perf_counter()
    e0.record()
    for _ in range(steps):
        step(mark=True)
    e1.record()
    host_ms = (time.perf_counter() - t0) * 1e3 / steps
    torch.cuda.synchronize()
    status = B.mohge_get_device_status(buf.ws)
    ms = e0.elapsed_time(e1) / steps
    gemm_ms = sum(a.elapsed_time(b) + c.elapsed_time(d_) for a, b, c, d_ in marks) / len(marks)
    counts = buf.counts.cpu().tolist()
    tf = flops_per_step(wl, counts) / (gemm_ms * 1e-3) / 1e12
    bf16 = wl.dtype == "bf16"
    return {"workload": wl.name, "dtype": wl.dtype, "T": wl.T, "steps": steps, "value": wl.T / (ms * 1e-3),
            "unit": UNIT, "ms_per_step": ms, "host_enqueue_ms_per_step": host_ms,
            "gemm_ms_per_step": gemm_ms, "gemm_tflops": tf,
            "gemm_frac_of_sustained_bf16": tf / pk["tf_sustained"] if bf16 else None,
            "count_ratio": count_ratio(counts), "device_status": status}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=list(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip what the default line adds outside the timed region: the per-step "
                         "HBM rooflines and the short runs of the other benchmark workloads")
    ap.add_argument("--forward-only", action="store_true",
                    help="time the forward pass alone (inference-shaped workloads); the roofline "
                         "object then describes mohge_expert_fwd against HBM bandwidth")
    ap.add_argument("--shared-width", type=int, default=0,
                    help="hidden width of the shared experts (N_s FFNs concatenated); 0 = none, "
                         "the benchmark configurations have none")
    ap.add_argument("--gather", action="store_true",
                    help="time the route that never writes x_perm (mohge_dispatch_indices, "
                         "mohge_expert_fwd_gather, mohge_expert_bwd_gather); BF16 workloads only")
    ap.add_argument("--dy-fused", action="store_true",
                    help="time the backward that never writes dy_perm (mohge_row_tokens, "
                         "mohge_expert_bwd_dy instead of mohge_combine_bwd, mohge_expert_bwd_dgate); "
                         "BF16 workloads only")
    ap.add_argument("--graph", action="store_true",
                    help="capture one step in a CUDA graph and time its replays (launch-bound small "
                         "workloads); the GEMM share for the roofline object is then taken from a "
                         "short eager loop before the timed region")
    args = ap.parse_args()
    if args.gather and args.dy_fused:
        ap.error("--gather and --dy-fused are separate routes: the backward without dy_perm reads x_perm")
    if args.forward_only:          # the end-to-end and CPU arms describe the fwd+bwd step only
        args.no_e2e = args.no_cpu_baseline = True
    wl = WORKLOADS[args.workload]
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, wl, rank)
        return

    from paper_2604_23108_b200 import binding as B
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    dist = None
    if world > 1:
        import torch.distributed as dist_
        dist = dist_
        dist.init_process_group("nccl", device_id=dev)

    gcfg = B.Config(d_model=wl.d_model, n_groups=wl.n_groups, experts_per_group=wl.experts_per_group,
                    k_groups=wl.k_groups, k_experts=wl.k_experts, group_width=list(wl.group_width),
                    dtype=wl.dtype, row_align=128 if wl.dtype == "bf16" else 1)
    inp = make_device_inputs(wl, dev, seed=replica_seed(wl, rank))
    buf = B.LayerBuffers(gcfg, wl.T, device=dev, shared_width=args.shared_width)
    shared = None
    if args.shared_width:
        from paper_2604_23108_b200.inputs import make_shared_weights
        shared = make_shared_weights(wl, args.shared_width, device=dev, seed=replica_seed(wl, rank))
    T = wl.T
    ev = lambda: torch.cuda.Event(enable_timing=True)
    if args.dy_fused:
        buf.hs = torch.empty_like(buf.h)
        buf.row_gate = torch.empty(buf.h.shape[0], dtype=torch.float32, device=buf.h.device)
    step, gemm_marks = make_step(B, gcfg, T, inp, buf, shared, args.shared_width, args.forward_only,
                                 args.gather, args.dy_fused)

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(3, args.warmup)):
        step()
    torch.cuda.synchronize()
    status = B.mohge_get_device_status(buf.ws)
    if status != 0:
        raise SystemExit("device status word = 0x%x after warm-up" % status)
    counts = buf.counts.cpu().tolist()

    graph = None
    if args.graph:
        # every launch of the step depends on device data only through device memory, so one
        # capture serves every later batch written into the same buffers
        for _ in range(min(args.steps, 10)):
            step(mark=True)
        torch.cuda.synchronize()
        l0 = B.mohge_launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            step()
        launches_per_replay = B.mohge_launch_count() - l0
        for _ in range(3):
            graph.replay()

    sampler = ClockSampler(local_rank) if rank == 0 else None
    l0 = B.mohge_launch_count()
    barrier()
    # host time to enqueue one step, taken on an empty launch queue (inside the timed loop of a
    # large workload the host mostly waits for room in the queue)
    host_t0 = time.perf_counter()
    for _ in range(3):
        if graph is not None:
            graph.replay()
        else:
            step()
    host_enqueue_ms = (time.perf_counter() - host_t0) * 1e3 / 3
    barrier()
    l0 = B.mohge_launch_count()
    t_start, t_end = ev(), ev()
    t_start.record()
    for _ in range(args.steps):
        if graph is not None:
            graph.replay()
        else:
            step(mark=True)
    t_end.record()
    barrier()
    launches = launches_per_replay * args.steps if graph is not None else B.mohge_launch_count() - l0
    clocks = sampler.stop() if sampler else None
    ms_total = t_start.elapsed_time(t_end)
    ms_total = max_over_ranks(ms_total, dist, dev)
    ms_step = ms_total / args.steps
    value = world * T / (ms_step * 1e-3)
    gemm_ms = [a.elapsed_time(b) + c.elapsed_time(d_) for a, b, c, d_ in gemm_marks]
    gemm_ms_step = sum(gemm_ms) / len(gemm_ms)

    # ---- end to end: host (pinned) inputs in, results back to the host, every step ----
    # A user of the library overlaps the copies with the kernels: three streams (upload, layer,
    # download) and two sets of device input/output buffers, ordered by events.  Every step
    # still uploads its own x and dy from pinned host memory and downloads its own y, dx and
    # losses; the timed region covers all of it.
    e2e = None
    if not args.no_e2e:
        hx = inp["x"].cpu().pin_memory()
        hdy = inp["dy"].cpu().pin_memory()
        hy = [torch.empty_like(hx).pin_memory() for _ in range(2)]
        hdx = [torch.empty_like(hx).pin_memory() for _ in range(2)]
        hloss = [torch.empty(4, dtype=torch.float32).pin_memory() for _ in range(2)]
        dx_in = [inp["x"], torch.empty_like(inp["x"])]
        ddy_in = [inp["dy"], torch.empty_like(inp["dy"])]
        dy_out = [torch.empty_like(buf.y) for _ in range(2)]
        ddx_out = [torch.empty_like(buf.dx) for _ in range(2)]
        dloss_out = [torch.empty_like(buf.loss) for _ in range(2)]
        s_up, s_down, s_main = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.current_stream()
        x_done = [torch.cuda.Event() for _ in range(2)]
        dy_done = [torch.cuda.Event() for _ in range(2)]
        in_free = [torch.cuda.Event() for _ in range(2)]
        y_ready = [torch.cuda.Event() for _ in range(2)]
        out_ready = [torch.cuda.Event() for _ in range(2)]
        out_free = [torch.cuda.Event() for _ in range(2)]
        for e_ in in_free + out_free:
            e_.record(s_main)

        def e2e_step(i):
            k = i & 1
            with torch.cuda.stream(s_up):
                s_up.wait_event(in_free[k])
                dx_in[k].copy_(hx, non_blocking=True)
                x_done[k].record(s_up)                         # the forward needs x only
                ddy_in[k].copy_(hdy, non_blocking=True)
                dy_done[k].record(s_up)
            s_main.wait_event(x_done[k])
            inp["x"], inp["dy"] = dx_in[k], ddy_in[k]
            s_main.wait_event(out_free[k])

            def after_fwd():                                   # y goes home while the backward runs
                y_ready[k].record(s_main)
                with torch.cuda.stream(s_down):
                    s_down.wait_event(y_ready[k])
                    hy[k].copy_(dy_out[k], non_blocking=True)

            step(y=dy_out[k], dx=ddx_out[k], after_fwd=after_fwd,      # y and dx go to this step's
                 before_bwd=lambda: s_main.wait_event(dy_done[k]))     # own set of buffers
            in_free[k].record(s_main)
            dloss_out[k].copy_(buf.loss, non_blocking=True)
            out_ready[k].record(s_main)
            with torch.cuda.stream(s_down):
                s_down.wait_event(out_ready[k])
                hdx[k].copy_(ddx_out[k], non_blocking=True)
                hloss[k].copy_(dloss_out[k], non_blocking=True)
                out_free[k].record(s_down)

        e2e_step(0)
        e2e_step(1)
        barrier()
        s0, s1 = ev(), ev()
        n_e2e = max(4, args.steps)      # as many steps as the device-only arm: the first upload and the
                                        # last download are inside the timed region and overlap nothing
        s0.record()
        for i in range(n_e2e):
            e2e_step(i)
        s_main.wait_stream(s_down)
        s_main.wait_stream(s_up)
        s1.record()
        barrier()
        ms = s0.elapsed_time(s1)
        inp["x"], inp["dy"] = dx_in[0], ddy_in[0]
        # what came back to the host is the layer's result: every step had the same inputs and the
        # layer is run-to-run bit-identical, so the last download must equal a device-only step
        step()
        torch.cuda.synchronize()
        last = (n_e2e - 1) & 1
        if not (torch.equal(hy[last], buf.y.cpu()) and torch.equal(hdx[last], buf.dx.cpu())
                and torch.equal(hloss[last][:buf.loss.numel()], buf.loss.cpu())):
            raise SystemExit("end-to-end arm: downloaded results differ from the device-only step")
        ms = max_over_ranks(ms, dist, dev)
        es = hx.element_size()
        e2e = {"value": world * T / (ms / n_e2e * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": 2 * hx.numel() * es,
               "d2h_bytes_per_step": 2 * hx.numel() * es + 16,
               "overlap": "uploads and downloads on their own streams, double-buffered; the forward "
                          "starts when x has arrived, y leaves while the backward runs",
               "checked": "last download equals a device-only step bit for bit"}

    status = B.mohge_get_device_status(buf.ws)
    if status != 0:
        raise SystemExit("device status word = 0x%x after the timed region" % status)

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    pk = _peaks()
    # ---- outside the timed region: every HBM-bound entry point on its own, then short runs of the
    # other benchmark workloads (default line only) ----
    hbm_steps, others = None, None
    if not args.no_extras and world == 1 and not args.forward_only and not args.shared_width and not args.gather \
            and not args.dy_fused:
        hbm_steps = hbm_step_rooflines(B, gcfg, wl, inp, buf, pk["hbm"])
        if args.workload == DEFAULT_WORKLOAD:
            others = [quick_workload_line(B, n, dev, pk) for n in
                      ("cfg1_tiny_f32", "cfg2_bf16", "cfg3_bf16_aux", "cfg4_bf16_skew")]
    flops = flops_per_step(wl, counts, args.shared_width)
    achieved = flops / (gemm_ms_step * 1e-3) / 1e12
    roofline = {"bound": "tensor", "achieved": achieved, "peak": pk["tf_sustained"], "unit": "TFLOP/s",
                "frac": achieved / pk["tf_sustained"], "traffic": NCU_DRAM_TRAFFIC_PER_STEP.get(wl.name),
                "traffic_unit": "bytes of DRAM traffic per step (six launches)",
                "traffic_source": NCU_DRAM_TRAFFIC_SOURCE.get(wl.name),
                "kernel": "tc_grouped_kernel (6 launches per step: fwd1, fwd2, dgrad x2, wgrad x2)",
                "of": pk["source"], "flops_per_step": flops, "gemm_ms_per_step": gemm_ms_step,
                "frac_of_nominal_2250": achieved / 2250.0}
    if args.forward_only:
        # expert forward of a small batch: what has to move is the weights of the experts that
        # were hit (read once), their rows of x_perm and the saved A, U, H and y_perm rows
        es = 2 if wl.dtype == "bf16" else 4
        N = wl.experts_per_group
        wbytes = sum(3 * wl.d_model * wl.group_width[e // N] * es for e, m in enumerate(counts) if m > 0)
        rbytes = sum(m * (2 * wl.d_model + 3 * wl.group_width[e // N]) * es for e, m in enumerate(counts))
        gbs = (wbytes + rbytes) / (gemm_ms_step * 1e-3) / 1e9
        roofline = {"bound": "hbm", "achieved": gbs, "peak": pk["hbm"], "unit": "GB/s",
                    "frac": gbs / pk["hbm"], "traffic": None,
                    "kernel": "tc_grouped_kernel (2 launches per step: fwd1, fwd2)", "of": pk["source"],
                    "bytes_per_step": wbytes + rbytes, "expert_fwd_ms_per_step": gemm_ms_step}
    if wl.dtype != "bf16":
        roofline.update(bound="alu", peak=None, frac=None,
                        kernel="simt_grouped_kernel (FP32 FMA; correctness configuration)")
    cpu_baseline = None
    if not args.no_cpu_baseline and world == 1:      # timed at N = 1 only: the other GPUs would wait
        from paper_2604_23108_b200.inputs import make_inputs
        sample = min(wl.T, ORACLE_SAMPLE_TOKENS)
        val, per, n, t_conv = oracle_sample_run(wl, sample, 1, 0, inp_cpu=make_inputs(wl, T=sample))
        cpu_baseline = oracle_baseline_dict(val, per, n, t_conv, sample, torch.get_num_threads())
    line = {
        "metric": METRIC_FWD if args.forward_only else METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(3, args.warmup), "ms_per_step": ms_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": wl.dtype, "data": "synthetic",
        "config": {"workload": wl.name, "T": T, "d_model": wl.d_model, "n_groups": wl.n_groups,
                   "experts_per_group": wl.experts_per_group, "group_width": list(wl.group_width),
                   "k_groups": wl.k_groups, "k_experts": wl.k_experts, "shared_width": args.shared_width,
                   "pass": "forward only" if args.forward_only else "forward + backward",
                   "count_ratio": count_ratio(counts),
                   "l2": "inputs larger than L2 (no flush)", "parallelism": "replicas only",
                   "launch": "CUDA graph replay" if args.graph else "stream launches",
                   "x_perm": "never written (rows gathered by the GEMMs)" if args.gather else "materialised",
                   "dy_perm": "never written (rows gathered by the GEMMs)" if args.dy_fused else "materialised"},
        "clocks": clocks, "e2e": e2e, "gpu_launches": launches, "device_status": status,
        "host_enqueue_ms_per_step": host_enqueue_ms,
        "roofline": roofline, "roofline_hbm_steps": hbm_steps, "cpu_baseline": cpu_baseline,
        "other_workloads": others,
    }
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
