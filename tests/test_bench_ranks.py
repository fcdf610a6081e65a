"""The N > 1 path of bench.py on CPU: two gloo ranks agree on the max-over-ranks step time, the
whole-job value counts every rank's bytes, and the reference arm prints on rank 0 only."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _rank_main(rank, world, port, out):
    sys.path.insert(0, ROOT)
    import bench
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ms = bench.reduce_max(10.0 + 5.0 * rank, world, torch.device("cpu"))
    dist.barrier()
    out[rank] = (ms, bench.aggregate_gbs(1_000_000_000, world, ms))
    dist.destroy_process_group()


def test_two_gloo_ranks_agree_on_max_time_and_aggregate_value():
    world = 2
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_rank_main, args=(world, 29613, out), nprocs=world, join=True)
        res = dict(out)
    assert res[0] == res[1]
    ms, gbs = res[0]
    assert ms == 15.0                                   # the slower rank
    assert abs(gbs - 2 * 1.0 / 15e-3) < 1e-9            # two ranks' bytes over the max time


def test_reference_arm_prints_on_rank_zero_only():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29614", os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
           "--workload", "fc", "--steps", "1", "--warmup", "0"]
    res = subprocess.run(cmd, capture_output=True, text=True, env=env, cwd=ROOT, timeout=300)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["cpu_baseline"]["kind"] == "oracle"
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["value"] > 0
