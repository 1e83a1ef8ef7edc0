"""The N > 1 path of bench.py on CPU: two gloo ranks.  The path has no exchange step
(every rank is an independent replica), so what the ranks share is the launch
environment, the max-over-ranks timing and the rule that rank 0 alone reports."""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def torchrun(nproc, script_args, timeout=300):
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port())] + script_args
    env = dict(os.environ, OMP_NUM_THREADS="2")
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


WORKER = r'''
import os, sys
sys.path.insert(0, os.getcwd())
import torch, torch.distributed as dist
import bench
rank, world, local = bench.dist_env()
assert world == 2 and rank == local and rank in (0, 1)
dist.init_process_group("gloo")
# each rank times its own replica; the job takes as long as the slowest one
mine = 10.0 + 5.0 * rank
slowest = bench.max_over_ranks(mine, world, device="cpu")
assert slowest == 15.0, slowest
# weak scaling: both ranks did the same work in that time
assert abs(bench.job_throughput(world, 3e12, slowest) - 2 * 3e12 / 15e-3 / 1e12) < 1e-9
assert bench.max_over_ranks(7.0, 1, device="cpu") == 7.0
dist.barrier()
dist.destroy_process_group()
if rank == 0:
    print("RANK0-OK")
'''


def test_max_over_ranks_and_job_throughput_on_two_gloo_ranks(tmp_path):
    w = tmp_path / "worker.py"
    w.write_text(WORKER)
    r = torchrun(2, [str(w)])
    assert r.returncode == 0, r.stderr[-2000:]
    assert r.stdout.count("RANK0-OK") == 1


def test_reference_arm_under_torchrun_prints_one_line_from_rank_0():
    r = torchrun(2, ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
                     "--ref-seconds", "0.5"])
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    line = json.loads(lines[0])
    assert line["impl"] == "reference" and line["n_gpus"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
