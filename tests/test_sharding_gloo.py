"""The N > 1 path on CPU: two gloo ranks take coordinate shards (host logic of bench.py --gpus N).

Each rank runs the float64 oracle on its shard with the shard's global column offset; gathered, the shards
must equal the single-process run bit for bit (the step has no exchange between coordinates), per-shard
consensus errors must add up, and the timing reduction must return the slowest rank's time on every rank.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import detag_oracle as orc
from paper_2006_08085_b200 import inputs, sharding


def test_shard_bounds_cover_and_align():
    for d, world in ((10, 2), (4096, 2), (25_600_000, 8), (7, 4), (270_000, 3)):
        cuts = [sharding.shard_bounds(d, r, world) for r in range(world)]
        assert cuts[0][0] == 0 and cuts[-1][1] == d
        for (a0, a1), (b0, b1) in zip(cuts, cuts[1:]):
            assert a1 == b0 and a0 <= a1
        assert all(j0 % 4 == 0 for j0, j1 in cuts if j1 > j0)
    assert sharding.weak_scaling_offset(1000, 3) == 3000


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, d, steps, out_dir):
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        cfg = inputs.CONFIGS["cfg1"].with_d(d)
        m = inputs.gossip_matrix(cfg)
        eta = orc.spectrum(m.to_dense()).eta
        j0, j1 = sharding.shard_bounds(cfg.d, rank, world)
        a, c, x0 = inputs.objective_data(cfg, j0, j1)
        p = orc.Problem(m.row_ptr, m.col_idx, m.vals, cfg.K, eta, cfg.alpha, a, c, cfg.sigma, cfg.seed, j0)
        s = orc.run(p, x0, steps)
        ce = sharding.reduce_sum(orc.consensus_error(s.x), dist)
        slowest = sharding.reduce_max(10.0 + rank, dist)
        np.savez(os.path.join(out_dir, f"rank{rank}.npz"), x=s.x, y=s.y, g=s.g_new, ce=ce, slowest=slowest, j0=j0, j1=j1)
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_reproduce_the_single_process_run(tmp_path):
    world, d, steps = 2, 1001, 4
    mp.start_processes(_worker, args=(world, _free_port(), d, steps, str(tmp_path)), nprocs=world, join=True,
                       start_method="spawn")
    cfg = inputs.CONFIGS["cfg1"].with_d(d)
    m = inputs.gossip_matrix(cfg)
    a, c, x0 = inputs.objective_data(cfg)
    p = orc.Problem(m.row_ptr, m.col_idx, m.vals, cfg.K, orc.spectrum(m.to_dense()).eta, cfg.alpha, a, c, cfg.sigma,
                    cfg.seed, 0)
    full = orc.run(p, x0, steps)
    parts = [np.load(tmp_path / f"rank{r}.npz") for r in range(world)]
    assert [int(q["j0"]) for q in parts] == [0, 504] and int(parts[-1]["j1"]) == d
    assert np.array_equal(np.concatenate([q["x"] for q in parts], axis=1), full.x)
    assert np.array_equal(np.concatenate([q["y"] for q in parts], axis=1), full.y)
    assert np.array_equal(np.concatenate([q["g"] for q in parts], axis=1), full.g_new)
    for q in parts:
        assert float(q["ce"]) == pytest.approx(orc.consensus_error(full.x), rel=1e-12)
        assert float(q["slowest"]) == 11.0


def test_bench_starts_its_own_ranks_when_no_launcher_is_around():
    """`python bench.py --gpus 2` with WORLD_SIZE unset must start two ranks itself.  --host-only keeps the run on
    the CPU: the ranks meet over gloo and reduce the two scalars of the real run through the same helpers."""
    import json
    import subprocess
    import sys

    from conftest import ROOT

    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--host-only", "--config", "cfg2"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [json.loads(ln) for ln in res.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1  # rank 0 alone prints
    line = lines[0]
    assert line["host_only"] is True and line["n_gpus"] == 2
    assert line["slowest"] == 2.0  # MAX over ranks of (1 + rank)
    assert line["offset_sum"] == float(inputs.CONFIGS["cfg2"].d)  # rank 1's shard starts where rank 0's ends
