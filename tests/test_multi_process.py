"""The N > 1 path of the benchmark on CPU: the hot path does not shard (one GEMM, one GPU), so
`bench.py --gpus N` runs N independent replicas.  What the ranks share is the timing protocol
(barrier, maximum over ranks, whole-job value) and, for the reference arm, the rule that rank 0
alone runs and prints.  Both are exercised here with world_size 2 on the gloo backend."""
import json
import os
import socket
import subprocess
import sys

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    import bench
    my_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    dist.barrier()
    slowest = bench.max_over_ranks(my_ms, dist, "cpu")
    value = bench.replicas_value(1000.0, world, slowest * 1e-3)
    alone = bench.max_over_ranks(my_ms, None, "cpu")
    with open(os.path.join(out_dir, f"rank{rank}.json"), "w") as f:
        json.dump({"slowest": slowest, "value": value, "alone": alone}, f)
    dist.barrier()
    dist.destroy_process_group()


def test_max_over_ranks_and_whole_job_value_with_two_gloo_ranks(tmp_path):
    world, port = 2, free_port()
    mp.spawn(_rank_main, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    got = [json.load(open(tmp_path / f"rank{r}.json")) for r in range(world)]
    for r, g in enumerate(got):
        assert g["slowest"] == 15.0                       # every rank reports the slowest rank's time
        assert g["value"] == pytest.approx(2 * 1000.0 / 15e-3)   # units of all ranks / that time
        assert g["alone"] == 10.0 + 5.0 * r               # without a process group the value is the rank's own


def test_reference_arm_under_torchrun_runs_on_rank_zero_only():
    """`bench.py --impl reference` launched as two ranks: rank 0 times the oracle and prints the one
    JSON line, the other rank exits 0 without work."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()),
           os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
           "--ref-macs", "2e7"]
    env = dict(os.environ, OMP_NUM_THREADS="2")
    p = subprocess.run(cmd, capture_output=True, text=True, timeout=600, cwd=ROOT, env=env)
    assert p.returncode == 0, p.stderr[-2000:]
    lines = [ln for ln in p.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1, p.stdout
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["steps"] == 1
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
