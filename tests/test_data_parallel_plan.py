"""Host side of the data-parallel step on CPU: the slot arithmetic of ShardPlan, alone and across two gloo ranks.

The ranks convert their weight shards (the oracle stands in for the kernels here), all-gather the slots exactly as
the device path does, and must end up with the byte-identical conversion of the whole weight; the WGRAD sum is
exchanged the same way and every rank must end up with its own rows of the whole product."""
import json
import os
import socket
import subprocess
import sys

import numpy as np
import pytest

import oracle as orc
from paper_2506_08027_b200.dp import ShardPlan

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_plan_slots_tile_the_gathered_buffers():
    for world in (1, 2, 4, 8):
        plans = [ShardPlan(world, r, 256, 384, 128 * world * 3) for r in range(world)]
        p0 = plans[0]
        assert [p.rows() for p in plans] == [(r * p0.F_r, (r + 1) * p0.F_r) for r in range(world)]
        for nbytes, total in ((p0.q_slot_bytes, p0.F * p0.H), (p0.s_row_slot_bytes, p0.s_row_bytes), (p0.s_col_part_bytes, p0.s_col_bytes)):
            edges = [p.slot(nbytes) for p in plans]
            assert edges[0][0] == 0 and edges[-1][1] == total
            assert all(edges[r][1] == edges[r + 1][0] for r in range(world - 1))
        assert sorted(p.first_owner() for p in plans) == list(range(world))    # ranks start at different owners
    # sizes agree with the layout formula of the library's scale arrays
    p = ShardPlan(2, 1, 128, 256, 512)
    assert p.s_row_bytes == orc.swizzle_scales(np.zeros((512, 8), np.uint8)).size
    assert p.s_col_part_bytes == orc.swizzle_scales(np.zeros((256, 8), np.uint8)).size


@pytest.mark.parametrize("args", [(0, 0, 128, 128, 128), (2, 2, 128, 128, 256), (9, 0, 128, 128, 9 * 128), (2, 0, 100, 128, 256),
                                  (2, 0, 128, 100, 256), (2, 0, 128, 128, 384), (4, 0, 128, 128, 256)])
def test_plan_refuses_shapes_the_kernels_cannot_shard(args):
    with pytest.raises(ValueError):
        ShardPlan(*args)


WORKER = r'''
import os, sys, json
sys.path.insert(0, os.environ["REPO_ROOT"]); sys.path.insert(0, os.path.join(os.environ["REPO_ROOT"], "tests"))
import numpy as np, torch, torch.distributed as dist
import oracle as orc
from paper_2506_08027_b200 import synth
from paper_2506_08027_b200.dp import ShardPlan
rank = int(os.environ["RANK"]); world = int(os.environ["WORLD_SIZE"])
dist.init_process_group("gloo", rank=rank, world_size=world)
T, H, F = 128, 128, 512
plan = ShardPlan(world, rank, T, H, F)
w = orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(0.02 * synth.gaussian((F, H), 41)))
lo, hi = plan.rows()
mine = w[lo:hi]
# the rank's conversions go into its slots of the gathered buffers
bufs = {"q_row": np.zeros(F * H, np.uint8), "q_col": np.zeros(F * H, np.uint8),
        "s_row": np.zeros(plan.s_row_bytes, np.uint8), "s_col_parts": np.zeros(plan.s_col_bytes, np.uint8)}
slot = {"q_row": plan.q_slot_bytes, "q_col": plan.q_slot_bytes, "s_row": plan.s_row_slot_bytes, "s_col_parts": plan.s_col_part_bytes}
qr, sr = orc.quantize(mine, orc.ROW); qc, sc = orc.quantize(mine, orc.COL)
own = {"q_row": qr.reshape(-1), "q_col": qc.reshape(-1), "s_row": orc.swizzle_scales(sr),
       "s_col_parts": orc.swizzle_scales(np.ascontiguousarray(sc.T))}
for k in bufs:
    a, b = plan.slot(slot[k]); bufs[k][a:b] = own[k]
    full = torch.from_numpy(bufs[k]); parts = list(full.view(world, -1).unbind(0))
    dist.all_gather(parts, full[a:b].clone())          # slot r of every rank, in rank order, in place
s_col = orc.concat_swizzled_scales_k([bufs["s_col_parts"][r * plan.s_col_part_bytes:(r + 1) * plan.s_col_part_bytes] for r in range(world)],
                                     H, plan.F_r // 32)
fq_r, fs_r = orc.quantize(w, orc.ROW); fq_c, fs_c = orc.quantize(w, orc.COL)
ok = (np.array_equal(bufs["q_row"], fq_r.reshape(-1)) and np.array_equal(bufs["q_col"], fq_c.reshape(-1))
      and np.array_equal(bufs["s_row"], orc.swizzle_scales(fs_r)) and np.array_equal(s_col, orc.swizzle_scales(np.ascontiguousarray(fs_c.T))))
# WGRAD: every rank's partial product over its own tokens, summed, each rank keeping its rows
x = orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(synth.gaussian((T, H), 50 + rank)))
dy = orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(synth.output_gradient((T, F), 60 + rank)))
xq, dyq = orc.quantize(x, orc.COL), orc.quantize(dy, orc.COL)
part, _ = orc.gemm_f64(dyq[0], dyq[1], xq[0], xq[1], "mn", "mn")
total = torch.from_numpy(part.copy()); dist.all_reduce(total)
kept = total.numpy()[lo:hi]
xs = [orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(synth.gaussian((T, H), 50 + r))) for r in range(world)]
dys = [orc.bf16_bits_to_f32(synth.f32_to_bf16_bits(synth.output_gradient((T, F), 60 + r))) for r in range(world)]
_, _, want, sabs = orc.data_parallel_linear_f64(xs, [w[plan.rows(r)[0]:plan.rows(r)[1]] for r in range(world)], dys)
ok_dw = bool(np.abs(kept - want[rank]).max() <= 1e-13 * sabs[2][rank].max())
dist.barrier()
print(json.dumps({"rank": rank, "weight": bool(ok), "dw": ok_dw}), flush=True)
dist.destroy_process_group()
'''


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_two_gloo_ranks_assemble_the_whole_weight_and_their_rows_of_dw():
    orc.build_oracle()          # once, before the ranks start
    port = _free_port()
    procs = []
    for r in range(2):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE="2", MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), REPO_ROOT=ROOT)
        procs.append(subprocess.Popen([sys.executable, "-c", WORKER], env=env, stdout=subprocess.PIPE, stderr=subprocess.PIPE, text=True, cwd=ROOT))
    for r, p in enumerate(procs):
        out, err = p.communicate(timeout=300)
        assert p.returncode == 0, err[-3000:]
        got = json.loads(out.strip().splitlines()[-1])
        assert got == {"rank": r, "weight": True, "dw": True}
