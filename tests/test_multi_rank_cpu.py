"""The N > 1 path of the benchmark is "replicas only": every rank runs its own games, nothing is
exchanged inside a step, and the only cross-rank traffic is the barrier and the reductions around
the timed region.  These tests run that plumbing with two gloo ranks on the CPU."""
import json
import os
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

_WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["SPIRAL_ROOT"])
import torch
import bench
world, rank, local = bench.dist_setup(2)
assert world == 2 and rank in (0, 1)
bench.barrier(world)
dev = torch.device("cpu")
# the slowest rank sets the time; the token counts add up
t = bench.max_over_ranks(10.0 + 5.0 * rank, world, dev)
n = bench.sum_over_ranks(128.0 * 7, world, dev)
assert t == 15.0 and n == 2 * 128 * 7, (t, n)
bench.barrier(world)
import torch.distributed as dist
dist.destroy_process_group()
import sys
sys.stdout.write(f"rank {rank} ok\n")       # one write per rank: two ranks share the pipe
sys.stdout.flush()
"""


def _torchrun(args, env_extra=None, timeout=600):
    env = dict(os.environ)
    env["SPIRAL_ROOT"] = ROOT
    env["OMP_NUM_THREADS"] = "2"
    env.update(env_extra or {})
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "2", "--master-addr",
           "127.0.0.1", "--master-port", "29511"] + args
    return subprocess.run(cmd, cwd=ROOT, env=env, capture_output=True, text=True, timeout=timeout)


def test_two_gloo_ranks_reduce_time_and_tokens(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    r = _torchrun([str(script)])
    assert r.returncode == 0, r.stdout + r.stderr
    assert "rank 0 ok" in r.stdout and "rank 1 ok" in r.stdout


def test_reference_arm_under_two_ranks_prints_one_line():
    """`bench.py --impl reference` under torchrun: rank 0 alone times the oracle and prints the JSON
    line, the other rank exits 0 without work."""
    r = _torchrun([os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--workload", "tiny_4seqs",
                   "--steps", "3", "--warmup", "1"])
    assert r.returncode == 0, r.stdout + r.stderr
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1, r.stdout
    j = json.loads(lines[0])
    assert j["impl"] == "reference" and j["steps"] == 3 and j["value"] > 0
    assert j["cpu_baseline"]["kind"] == "oracle" and j["e2e"]["h2d_bytes_per_step"] == 0
