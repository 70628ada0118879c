"""The benchmark's N > 1 plumbing on CPU: two gloo ranks agree on the
max-over-ranks time and the summed token count, and the reference arm prints
from rank 0 only."""
import json
import os
import socket
import subprocess
import sys
from pathlib import Path

ROOT = Path(__file__).resolve().parent.parent

RANK_SCRIPT = r"""
import os, sys, json
sys.path.insert(0, os.environ["PAMM_ROOT"])
import bench
rank, world = bench.dist_setup(world_hint := 2, "gloo")
ms, tokens = bench.aggregate(10.0 + 5.0 * rank, 1000 * (rank + 1))
bench.barrier()
print(json.dumps({"rank": rank, "world": world, "ms": ms, "tokens": tokens}), flush=True)
import torch.distributed as dist
dist.destroy_process_group()
"""


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _env(rank: int, port: int) -> dict:
    env = dict(os.environ)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(port), PAMM_ROOT=str(ROOT))
    return env


def test_two_gloo_ranks_aggregate_max_time_and_sum_tokens():
    port = _free_port()
    procs = [subprocess.Popen([sys.executable, "-c", RANK_SCRIPT], env=_env(r, port), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=120)
        assert p.returncode == 0, err
        outs.append(json.loads(out.strip().splitlines()[-1]))
    assert {o["rank"] for o in outs} == {0, 1}
    for o in outs:
        assert o["world"] == 2
        assert o["ms"] == 15.0          # max over ranks
        assert o["tokens"] == 3000      # whole-job sum


def test_single_rank_aggregate_is_identity():
    sys.path.insert(0, str(ROOT))
    import bench
    assert bench.aggregate(3.5, 42) == (3.5, 42)


def test_reference_arm_prints_from_rank_zero_only():
    cmd = [sys.executable, str(ROOT / "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0",
           "--workload", "c1", "--ref-tokens", "512"]
    port = _free_port()
    r1 = subprocess.run(cmd, env=_env(1, port), capture_output=True, text=True, timeout=300)
    assert r1.returncode == 0 and r1.stdout.strip() == ""
    r0 = subprocess.run(cmd, env=_env(0, port), capture_output=True, text=True, timeout=300)
    assert r0.returncode == 0, r0.stderr
    line = json.loads(r0.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "tokens/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
