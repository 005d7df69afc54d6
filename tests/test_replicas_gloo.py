"""Host-side logic of the N > 1 path of bench.py, on CPU: two `gloo` ranks.

The view step does not shard (replicas only), so the multi-rank logic is: which view each replica renders, the
maximum-over-ranks timing, the whole-job value, and the reference arm printing on rank 0 only."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import json, os, sys
sys.path.insert(0, {root!r})
import torch
import torch.distributed as dist
import bench

rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
local_ms = 10.0 * (rank + 1)                      # rank 1 is the slow one
ms = bench.max_over_ranks(local_ms, world, torch.device("cpu"))
views = [bench.replica_view(s, rank, 8) for s in range(10)]
dist.barrier()
print(json.dumps({{"rank": rank, "ms": ms, "value": bench.whole_job_value(5, world, ms * 1e-3), "views": views}}))
dist.destroy_process_group()
"""


def free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def rank_env(rank: int, world: int, port: int) -> dict:
    env = dict(os.environ)
    env.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
               MASTER_PORT=str(port))
    return env


@pytest.mark.timeout(180)
def test_two_gloo_ranks_take_the_slowest_time_and_different_views():
    port = free_port()
    code = WORKER.format(root=ROOT)
    procs = [subprocess.Popen([sys.executable, "-c", code], env=rank_env(r, 2, port), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=170)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    outs.sort(key=lambda o: o["rank"])
    # both ranks agree on the slowest rank's time, and the value counts the views of both replicas
    assert outs[0]["ms"] == outs[1]["ms"] == 20.0
    assert outs[0]["value"] == outs[1]["value"] == pytest.approx(2 * 5 / 0.020)
    # replica r starts at view r: at every step the two replicas render different cameras
    assert outs[0]["views"] == [s % 8 for s in range(10)]
    assert outs[1]["views"] == [(s + 1) % 8 for s in range(10)]
    assert all(a != b for a, b in zip(outs[0]["views"], outs[1]["views"]))


@pytest.mark.timeout(300)
def test_reference_arm_under_two_ranks_prints_on_rank_zero_only():
    port = free_port()
    cmd = [sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--config", "1",
           "--steps", "2", "--warmup", "1"]
    procs = [subprocess.Popen(cmd, env=rank_env(r, 2, port), stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True,
                              cwd=ROOT) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=280)
        assert p.returncode == 0, err[-2000:]
        outs.append(out.strip())
    assert outs[1] == ""                                       # the other rank exits 0 without work
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["steps"] == 2
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["value"] == line["value"]
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0
    assert line["value"] > 0
