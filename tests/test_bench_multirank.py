"""The multi-rank plumbing of bench.py on CPU: two gloo ranks, no GPU.

Each rank of the benchmark processes its own batch (no collective on the data path); the only
exchange is the MAX of the device times.  Checked here: the slowest rank's time wins on every
rank, the whole-job value counts every rank's work, and the reference arm prints exactly one
line (rank 0) while the other rank exits quietly.
"""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r'''
import os, sys, json
sys.path.insert(0, os.environ["REPO_ROOT"])
import torch.distributed as dist
import bench
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
local_ms = 1.0 + 0.5 * rank            # rank 1 is the slow one
ms = bench.max_over_ranks(local_ms, world, "cpu")
val = bench.whole_job_value(world, ms)
dist.barrier()
print(json.dumps({"rank": rank, "ms": ms, "value": val}), flush=True)
dist.destroy_process_group()
'''


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _launch(rank, world, port, code=None, argv=None):
    env = dict(os.environ, RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
               MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), REPO_ROOT=ROOT)
    cmd = [sys.executable, "-c", code] if code else [sys.executable] + argv
    return subprocess.Popen(cmd, env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, cwd=ROOT)


def test_max_over_ranks_and_whole_job_value_with_two_gloo_ranks():
    port = _free_port()
    procs = [_launch(r, 2, port, code=WORKER) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=180)
        assert p.returncode == 0, err[-2000:]
        outs.append(json.loads(out.strip().splitlines()[-1]))
    import bench
    for o in outs:
        assert o["ms"] == pytest.approx(1.5)                       # the slow rank decides, on every rank
        assert o["value"] == pytest.approx(2 * bench.STEP_FLOP / 1.5e-3 / 1e12)
    assert bench.whole_job_value(1, 1.5) * 2 == pytest.approx(outs[0]["value"])


def test_reference_arm_prints_one_line_on_rank_zero_only():
    port = _free_port()
    argv = [os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1", "--warmup", "0"]
    procs = [_launch(r, 2, port, argv=argv) for r in range(2)]
    outs = []
    for p in procs:
        out, err = p.communicate(timeout=600)
        assert p.returncode == 0, err[-2000:]
        outs.append(out.strip())
    assert outs[1] == ""
    line = json.loads(outs[0].splitlines()[-1])
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["gpu_launches"] == 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["e2e"]["h2d_bytes_per_step"] == 0
    assert line["value"] > 0 and line["unit"] == "TFLOP/s"
