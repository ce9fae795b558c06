"""The multi-rank plumbing of bench.py on CPU: two gloo ranks, as torchrun would start them.

The path has no inter-GPU exchange (ranks are independent replicas), so the only collectives are the
barrier around the timed region and the max over ranks of the timed duration; the reference arm runs on
rank 0 alone.  Both are checked here without a GPU.
"""
import json
import os
import socket
import subprocess
import sys

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["REPO_ROOT"])
import bench
rank, world, local = bench.dist_setup(2)
assert world == 2 and rank == int(os.environ["RANK"]) and local == int(os.environ["LOCAL_RANK"])
bench.barrier(world)
slowest = bench.max_over_ranks(10.0 + 5.0 * rank, world, "cpu")     # rank 1 is the slower one
assert slowest == 15.0, slowest
bench.barrier(world)
import torch.distributed as dist
dist.destroy_process_group()
print("rank", rank, "ok")
"""


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _spawn(code_or_args, rank, port, extra_env=None):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(port), REPO_ROOT=ROOT, CUDA_VISIBLE_DEVICES="")
    env.update(extra_env or {})
    return subprocess.Popen([sys.executable] + code_or_args, env=env, cwd=ROOT, stdout=subprocess.PIPE,
                            stderr=subprocess.STDOUT, text=True)


def test_max_over_ranks_and_barrier_with_two_gloo_ranks():
    port = _free_port()
    procs = [_spawn(["-c", WORKER], r, port) for r in range(2)]
    outs = [p.communicate(timeout=180)[0] for p in procs]
    for r, (p, o) in enumerate(zip(procs, outs)):
        assert p.returncode == 0, o
        assert f"rank {r} ok" in o


def test_reference_arm_prints_on_rank_zero_only():
    port = _free_port()
    args = ["bench.py", "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0", "--workload", "c1"]
    procs = [_spawn(args, r, port) for r in range(2)]
    outs = [p.communicate(timeout=300)[0] for p in procs]
    assert procs[0].returncode == 0 and procs[1].returncode == 0, outs
    line = json.loads(outs[0].strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["cpu_baseline"]["kind"] == "oracle" and line["value"] > 0
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["gpu_launches"] == 0
    assert outs[1].strip() == ""                      # the other rank exits without work or output
