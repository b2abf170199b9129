"""Multi-rank host logic on CPU: world_size-2 gloo processes shard streams, gather results, reduce timings."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2402_04466_b200.sharding import assign_streams, gather_results, max_over_ranks, owner_of


def test_assignment_covers_every_stream_once():
    for n in range(0, 9):
        for w in (1, 2, 3, 4, 8):
            parts = assign_streams(n, w)
            flat = sorted(s for p in parts for s in p)
            assert flat == list(range(n))
            assert all(owner_of(s, w) == r for r, p in enumerate(parts) for s in p)
            assert max(len(p) for p in parts) - min(len(p) for p in parts) <= 1
    with pytest.raises(ValueError):
        assign_streams(3, 0)


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n_streams, out_dir):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = assign_streams(n_streams, world)[rank]
        local = {s: {"stream": s, "conf": [0.1 * s, 0.2 * s], "rank": rank} for s in mine}
        merged = gather_results(local, world)
        assert sorted(merged) == list(range(n_streams))
        assert all(merged[s]["rank"] == s % world and merged[s]["stream"] == s for s in merged)
        times = max_over_ranks([1.0 + rank, 5.0 - rank], world)
        assert times == [float(world), 5.0]
        dist.barrier()
        with open(os.path.join(out_dir, f"ok{rank}"), "w") as f:
            f.write("ok")
    finally:
        dist.destroy_process_group()


def test_two_rank_gather_and_timing_reduction(tmp_path):
    world, port = 2, _free_port()
    mp.spawn(_worker, args=(world, port, 5, str(tmp_path)), nprocs=world, join=True)
    assert all((tmp_path / f"ok{r}").exists() for r in range(world))
