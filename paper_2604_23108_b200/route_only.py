"""mohge_route alone at a workload's router shape, holding only the tensors that call needs
(x, the router weight, the outputs, the workspace: 0.7 GB at the large workload instead of the
45 GB of the whole layer), so that the routing kernel can be timed or profiled on its own.

    python -m paper_2604_23108_b200.route_only --workload cfg5_bf16_large [--calls 20] [--two-kernels]

Prints the time per call by CUDA events, the algorithmic bytes (x and the router weight read
once, every output written once) and the rate.  --two-kernels switches the selection in the
epilogue of the logits GEMM off (switch route_fused = 0): logits GEMM, then the selection kernel.
"""
from __future__ import annotations

import argparse

import torch

from . import binding as B
from .inputs import WORKLOADS


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--workload", default="cfg5_bf16_large", choices=list(WORKLOADS))
    ap.add_argument("--calls", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--two-kernels", action="store_true")
    args = ap.parse_args()
    wl = WORKLOADS[args.workload]
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(0)
    cfg = B.Config(d_model=wl.d_model, n_groups=wl.n_groups, experts_per_group=wl.experts_per_group,
                   k_groups=wl.k_groups, k_experts=wl.k_experts, group_width=list(wl.group_width),
                   dtype=wl.dtype)
    T, NL, Ne = wl.T, wl.n_logits, wl.n_experts
    dt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    g = torch.Generator(device=dev)
    g.manual_seed(wl.seed)
    x = torch.randn(T, wl.d_model, device=dev, generator=g).to(dt)
    w = (torch.randn(NL, wl.d_model, device=dev, generator=g) * 0.02).to(dt)
    logits = torch.empty(T, NL, device=dev)
    esp = torch.empty(T, Ne, device=dev)
    gs = torch.empty(T, wl.n_groups, device=dev)
    gi = torch.empty(T, wl.k_groups, dtype=torch.int32, device=dev)
    ei = torch.empty(T, wl.k_experts, dtype=torch.int32, device=dev)
    gw = torch.empty(T, wl.k_experts, device=dev)
    ws = torch.zeros(B.mohge_workspace_bytes(cfg, T), dtype=torch.uint8, device=dev)
    B.mohge_workspace_init(cfg, T, ws)
    if args.two_kernels:
        B.mohge_set_switch("route_fused", 0)

    def route():
        B.mohge_route(cfg, T, x, w, None, None, logits, gi, ei, gw, gs, esp, ws)

    n0 = B.mohge_launch_count()
    route()
    launches = B.mohge_launch_count() - n0
    for _ in range(args.warmup):
        route()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(args.calls):
        route()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / max(args.calls, 1)
    status = B.mohge_get_device_status(ws)
    nbytes = (x.numel() + w.numel()) * x.element_size() + 4 * (logits.numel() + esp.numel() + gs.numel()
                                                               + gi.numel() + ei.numel() + gw.numel())
    print("%s: mohge_route %.4f ms per call, %d launch(es), %.1f MB, %.0f GB/s, device status %d"
          % (wl.name, ms, launches, nbytes / 1e6, nbytes / ms / 1e6, status))
    if status != 0:
        raise SystemExit(1)


if __name__ == "__main__":
    main()
