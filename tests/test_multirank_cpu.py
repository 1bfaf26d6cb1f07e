"""World-size-2 gloo test (CPU) of the multi-GPU host logic: request sharding, max-over-ranks
timing, result gathering.  The data path has no collective, so this is all there is to cover."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_00938_b200.sharding import gather_results, max_over_ranks, request_shard


def test_request_shard_partitions_exactly():
    for n in (1, 7, 32, 33, 64):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen += list(request_shard(n, world, r))
            assert seen == list(range(n))
            sizes = [len(request_shard(n, world, r)) for r in range(world)]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out_dir):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = request_shard(5, world, rank)
        t = max_over_ranks(10.0 + rank)                 # rank 1 is slower: everyone must report 11.0
        local = torch.full((3,), float(rank)) + torch.tensor([len(mine), mine.start, 0.0])
        parts = gather_results(local)
        ok = (t == 11.0 and len(parts) == world and parts[0].tolist() == [3.0, 0.0, 0.0]
              and parts[1].tolist() == [3.0, 4.0, 1.0])
        with open(os.path.join(out_dir, f"rank{rank}.txt"), "w") as f:
            f.write("ok" if ok else f"bad t={t} parts={[p.tolist() for p in parts]}")
    finally:
        dist.destroy_process_group()


def test_two_ranks_gloo(tmp_path):
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    for r in range(2):
        assert open(tmp_path / f"rank{r}.txt").read() == "ok"
