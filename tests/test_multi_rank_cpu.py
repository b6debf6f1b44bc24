"""The N > 1 path on CPU: two gloo ranks.  The layer does not shard ("replicas only"), so what
several ranks share is the timing reduction (maximum over ranks), the per-rank seeds and the
rule that only rank 0 reports."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    from paper_2604_23108_b200.inputs import WORKLOADS, make_inputs
    wl = WORKLOADS["cfg1_tiny_f32"]
    slow = bench.max_over_ranks(10.0 + 5.0 * rank, dist, torch.device("cpu"))
    x = make_inputs(wl, seed=bench.replica_seed(wl, rank), weights=False)["x"]
    gathered = [torch.empty_like(x) for _ in range(world)]
    dist.all_gather(gathered, x)
    out[rank] = (slow, bool(torch.equal(gathered[0], gathered[1])))
    dist.destroy_process_group()


def test_max_over_ranks_and_independent_replica_batches():
    world, port = 2, 29000 + os.getpid() % 2000
    with mp.Manager() as m:
        out = m.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0][0] == res[1][0] == 15.0          # every rank sees the slowest rank's time
    assert res[0][1] is False and res[1][1] is False   # the replicas work on different batches
    import bench
    assert bench.max_over_ranks(3.5, None, torch.device("cpu")) == 3.5


def test_reference_arm_under_torchrun_prints_one_line_from_rank_zero():
    port = 31000 + os.getpid() % 2000
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(port), os.path.join(ROOT, "bench.py"),
           "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
           "--workload", "cfg1_tiny_f32"]
    r = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["value"] > 0 and d["e2e"]["h2d_bytes_per_step"] == 0
