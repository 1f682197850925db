"""The data-parallel linear step end to end: alone (one rank: must equal the single-device step bit for bit), and as
two processes that share one GPU, exchange the weight bytes through the host and add their WGRAD tiles into each
other's buffers through CUDA IPC mappings.  No kernel of one process waits for the other: the processes meet on
the host between launches only."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200 import synth

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _bf16(bits):
    import torch
    return torch.from_numpy(bits.view(np.int16)).cuda().view(torch.bfloat16)


@pytest.mark.parametrize("shape", [(128, 128, 128), (256, 384, 640), (1024, 512, 2048)])
def test_one_rank_equals_the_single_device_step(shape):
    import torch
    from paper_2506_08027_b200 import binding as B
    from paper_2506_08027_b200.dp import DataParallelLinear
    T, H, F = shape
    x = _bf16(synth.f32_to_bf16_bits(synth.gaussian((T, H), 5)))
    w = _bf16(synth.f32_to_bf16_bits(0.02 * synth.gaussian((F, H), 6)))
    dy = _bf16(synth.f32_to_bf16_bits(synth.output_gradient((T, F), 7)))
    y = torch.empty(T, F, dtype=torch.bfloat16, device="cuda")
    dx = torch.empty(T, H, dtype=torch.bfloat16, device="cuda")
    dw = torch.empty(F, H, dtype=torch.bfloat16, device="cuda")
    ws = torch.empty(B.mxfp8_linear_ws_bytes(T, H, F), dtype=torch.uint8, device="cuda")
    B.mxfp8_linear(x, w, dy, B.RULE_PAPER, y, dx, dw, ws)
    layer = DataParallelLinear(T, H, F)
    for _ in range(2):                                   # the second step starts from a used dW buffer
        before = B.mxfp8_launch_count()
        gy, gdx, gdw = layer.step(x, w, dy)
        assert B.mxfp8_launch_count() - before == 5     # cast W, cast X + dY, join scales, FPROP + DGRAD, WGRAD
        assert B.mxfp8_device_status() == 0
        assert torch.equal(gy.view(torch.int16), y.view(torch.int16))
        assert torch.equal(gdx.view(torch.int16), dx.view(torch.int16))
        assert torch.equal(gdw.to(torch.bfloat16).view(torch.int16), dw.view(torch.int16))   # FP32 here, BF16 (one rounding) there


def test_one_rank_group_runs_the_collectives_on_the_stream():
    """A one-rank NCCL group: the in-place all-gathers and the closing all-reduce are issued as on many GPUs."""
    import torch
    import torch.distributed as dist
    from paper_2506_08027_b200 import binding as B
    from paper_2506_08027_b200.dp import DataParallelLinear
    T, H, F = 256, 256, 384
    x = _bf16(synth.f32_to_bf16_bits(synth.gaussian((T, H), 15)))
    w = _bf16(synth.f32_to_bf16_bits(0.02 * synth.gaussian((F, H), 16)))
    dy = _bf16(synth.f32_to_bf16_bits(synth.output_gradient((T, F), 17)))
    alone = DataParallelLinear(T, H, F)
    want = [t.clone() for t in alone.step(x, w, dy)]
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    dist.init_process_group("nccl", init_method="tcp://127.0.0.1:%d" % port, rank=0, world_size=1)
    try:
        layer = DataParallelLinear(T, H, F, exchange_when_alone=True)
        assert layer.on_stream and layer.exchange
        for _ in range(2):
            got = layer.step(x, w, dy)
            torch.cuda.synchronize()
            assert B.mxfp8_device_status() == 0
            for g, t in zip(got, want):
                assert torch.equal(g, t)
    finally:
        dist.destroy_process_group()


WORKER = r'''
import os, sys, json
sys.path.insert(0, os.environ["REPO_ROOT"]); sys.path.insert(0, os.path.join(os.environ["REPO_ROOT"], "tests"))
import numpy as np, torch, torch.distributed as dist
import oracle as orc
from paper_2506_08027_b200 import synth, binding as B
from paper_2506_08027_b200.dp import DataParallelLinear
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
torch.cuda.set_device(0)
dist.init_process_group("gloo", rank=rank, world_size=world)
T, H, F = 256, 256, 512
def bits(a): return synth.f32_to_bf16_bits(a)
def dev(b): return torch.from_numpy(b.view(np.int16)).cuda().view(torch.bfloat16)
xb = [bits(synth.gaussian((T, H), 70 + r)) for r in range(world)]
dyb = [bits(synth.output_gradient((T, F), 80 + r)) for r in range(world)]
wb = bits(0.02 * synth.gaussian((F, H), 90))
layer = DataParallelLinear(T, H, F)
lo, hi = layer.plan.rows()
res = {}
for it in range(2):
    y, dx, dw = layer.step(dev(xb[rank]), dev(wb[lo:hi]), dev(dyb[rank]))
    torch.cuda.synchronize()
    assert B.mxfp8_device_status() == 0
    res[it] = (y.float().cpu().numpy().astype(np.float64), dx.float().cpu().numpy().astype(np.float64), dw.cpu().numpy().astype(np.float64))
f32 = orc.bf16_bits_to_f32
w = f32(wb)
ys, dxs, dws, (s_y, s_dx, s_dw) = orc.data_parallel_linear_f64([f32(b) for b in xb], [w[r * (F // world):(r + 1) * (F // world)] for r in range(world)],
                                                               [f32(b) for b in dyb])
def worst(got, want, sabs, bf16):
    bound = 2.0 ** -16 * sabs + (2.0 ** -8 * np.abs(want) if bf16 else 0) + 2.0 ** -126
    return float((np.abs(got - want) / bound).max())
out = {"rank": rank, "same_twice": all(np.array_equal(a, b) for a, b in zip(res[0], res[1])),
       "y": worst(res[1][0], ys[rank], s_y[rank], True), "dx": worst(res[1][1], dxs[rank], s_dx[rank], True),
       "dw": worst(res[1][2], dws[rank], s_dw[rank], False), "launches": int(B.mxfp8_launch_count())}
dist.barrier()
print(json.dumps(out), flush=True)
del layer
dist.destroy_process_group()
'''


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_processes_on_one_gpu_exchange_through_ipc_mappings():
    orc.build_oracle()          # once, before the ranks start
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), REPO_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, cwd=ROOT))
    for r, p in enumerate(procs):
        out, err = p.communicate(timeout=600)
        assert p.returncode == 0, err[-3000:]
        got = json.loads(out.strip().splitlines()[-1])
        assert got["rank"] == r and got["launches"] == 10
        assert got["same_twice"]                 # two contributions per element: the sum does not depend on arrival order
        assert got["y"] <= 1.0 and got["dx"] <= 1.0 and got["dw"] <= 1.0, got
