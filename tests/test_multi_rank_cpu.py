"""The N > 1 path on CPU: two gloo ranks shard rows with no data exchange, run the CPU oracle on
their shard (the stand-in for the per-rank device work), and reduce only their timing. CPU only."""
import os
import socket
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2607_24762_b200 import sharding  # noqa: E402


def test_row_shard_covers_without_overlap():
    for rows in (0, 1, 7, 64, 1000, 131072):
        for world in (1, 2, 3, 8):
            spans = [sharding.row_shard(rows, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == rows
            for (a, b), (c, d) in zip(spans, spans[1:]):
                assert b == c and a <= b and c <= d
            sizes = [b - a for a, b in spans]
            assert max(sizes) - min(sizes) <= 1
    with pytest.raises(ValueError):
        sharding.row_shard(10, 2, 2)


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, out_dir: str):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        from oracle import fso
        from paper_2607_24762_b200 import workloads as W
        w = W.WORKLOADS["cfg1"]
        lo, hi = sharding.row_shard(w.rows, rank, world)
        x = W.generate_rows(w, lo, hi)                       # each rank generates only its rows
        y = fso.softmax_f64(x, w.dtype, w.scale_f32)
        np.save(os.path.join(out_dir, f"y{rank}.npy"), y)
        # timing reduction: the job is as slow as its slowest rank
        mine = 1.0 + rank
        slowest = sharding.max_over_ranks(mine)
        assert slowest == float(world)
        assert sharding.aggregate_throughput(10.0, slowest, world) == 10.0 * world / world
        spans = [None] * world
        dist.all_gather_object(spans, (lo, hi))
        assert spans[0][0] == 0 and spans[-1][1] == w.rows and all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
        dist.barrier()
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_shard_rows_and_reduce_timing(tmp_path):
    world = 2
    mp.spawn(_worker, args=(world, _free_port(), str(tmp_path)), nprocs=world, join=True)
    from oracle import fso
    from paper_2607_24762_b200 import workloads as W
    w = W.WORKLOADS["cfg1"]
    whole = fso.softmax_f64(W.generate(w), w.dtype, w.scale_f32)
    parts = np.concatenate([np.load(tmp_path / f"y{r}.npy") for r in range(world)])
    assert np.array_equal(parts, whole)                      # sharding by rows changes nothing


def test_max_over_ranks_is_identity_without_a_group():
    assert sharding.max_over_ranks(3.5) == 3.5
