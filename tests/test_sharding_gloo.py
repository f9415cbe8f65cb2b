"""The multi-GPU story of this path is a partition with no exchange: every rank searches whole strips of
M-row multiples (or whole matrices) and only the scalar objective is summed.  This checks that host logic
with two gloo ranks on CPU (the per-rank search is done by the CPU oracle here; on GPUs each rank calls
tm_find_mask on its strip)."""
from __future__ import annotations

import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads
from oracle import tm_oracle as orc
from paper_2102_08124_b200.sharding import row_strip


def _free_port():
    s = socket.socket(); s.bind(("127.0.0.1", 0)); p = s.getsockname()[1]; s.close(); return p


def _worker(rank, world, port, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"; os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    W = workloads.normal_f32(72, 160, 0.02, 321)
    r0, r1 = row_strip(W.shape[0], 4, world, rank)
    res = orc.find_mask(np.ascontiguousarray(W[r0:r1]), 2, 4, orc.APPROX)
    obj = torch.tensor([res["objective"]], dtype=torch.float64)
    dist.all_reduce(obj, op=dist.ReduceOp.SUM)                   # the only cross-rank quantity
    t = torch.tensor([float(rank + 1)], dtype=torch.float64)     # stand-in for the per-rank device time
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    np.save(os.path.join(out_dir, "mask%d.npy" % rank), res["mask"])
    np.save(os.path.join(out_dir, "meta%d.npy" % rank), np.array([r0, r1, obj.item(), t.item()]))
    dist.barrier()
    dist.destroy_process_group()


def test_row_strips_cover_the_matrix_without_overlap():
    for rows, M, world in [(72, 4, 2), (8, 8, 4), (4, 4, 3), (0, 4, 2), (1024, 8, 8), (20, 4, 8)]:
        strips = [row_strip(rows, M, world, r) for r in range(world)]
        assert strips[0][0] == 0 and strips[-1][1] == rows
        for a, b in zip(strips, strips[1:]):
            assert a[1] == b[0]
        assert all(s[0] % M == 0 and s[1] % M == 0 and s[0] <= s[1] for s in strips)
        sizes = [(s[1] - s[0]) // M for s in strips]
        assert max(sizes) - min(sizes) <= 1


def test_two_ranks_reproduce_the_unsharded_result(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    W = workloads.normal_f32(72, 160, 0.02, 321)
    whole = orc.find_mask(W, 2, 4, orc.APPROX)
    parts = [np.load(tmp_path / ("mask%d.npy" % r)) for r in range(world)]
    metas = [np.load(tmp_path / ("meta%d.npy" % r)) for r in range(world)]
    assert np.array_equal(np.concatenate(parts, axis=0), whole["mask"])
    for m in metas:
        assert abs(m[2] - whole["objective"]) <= 1e-12 * whole["objective"]
        assert m[3] == float(world)                                # max over ranks


def test_bench_starts_its_own_ranks():
    """`bench.py --gpus 2` outside a torchrun environment starts two ranks itself (rendezvous on 127.0.0.1) and rank 0 prints
    one line that counts both; here with the GPU step replaced by the host stand-in of --dry-run (gloo)."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "4", "--warmup", "3", "--dry-run"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert out.returncode == 0, out.stderr[-2000:]
    lines = [ln for ln in out.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                                      # rank 0 alone prints
    line = json.loads(lines[0])
    assert line["n_gpus"] == 2 and line["steps"] == 4 and line["warmup"] == 3 and line["scaling"] == "weak"
