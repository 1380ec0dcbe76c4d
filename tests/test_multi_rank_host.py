"""The N > 1 path of the benchmark on CPU: ranks are independent replicas, the only cross-rank
steps are a barrier and a max over ranks of the measured time.  Run as two gloo processes."""
import json
import os
import socket
import subprocess
import sys


ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, %r)
import torch, torch.distributed as dist
import bench
dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
mine = 10.0 + 5.0 * rank                      # rank 1 is the slow replica
slowest = bench.max_over_ranks(mine, dist, world, "cpu")
assert slowest == 10.0 + 5.0 * (world - 1), slowest
v = bench.whole_job_gbs(4_000_000_000, 3, world, slowest)
assert abs(v - world * 4e9 * 3 / (slowest * 1e-3) / 1e9) < 1e-9
dist.barrier()
if rank == 0:
    print("OK", slowest, v)
dist.destroy_process_group()
"""


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _torchrun(args, timeout):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    return subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1",
                           "--nproc-per-node", "2", "--master-addr", "127.0.0.1",
                           "--master-port", str(_free_port())] + args,
                          cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_max_over_ranks_and_aggregate_with_two_gloo_ranks(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(WORKER % ROOT)
    r = _torchrun([str(script)], 240)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("OK")]
    assert lines == ["OK 15.0 1600.0"], r.stdout   # 2 ranks x 12 GB over 15 ms


def test_reference_arm_prints_one_line_from_rank0_under_two_ranks():
    r = _torchrun(["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"],
                  600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["n_gpus"] == 2 and d["value"] > 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["e2e"]["h2d_bytes_per_step"] == 0 and d["e2e"]["d2h_bytes_per_step"] == 0
