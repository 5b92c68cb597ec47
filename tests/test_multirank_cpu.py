"""Multi-rank host logic on CPU (gloo, world size 2): disjoint block ownership that covers the
cache, and the max-over-ranks reduction the benchmark uses for its timings."""
import os
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, out):
    sys.path.insert(0, ROOT)
    from paper_2605_02905_b200 import shard
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    blocks = shard.block_range(7, 4, rank, world)          # 7 streams of 4 blocks, keys and values
    owned = torch.zeros(7 * 8, dtype=torch.int64)
    owned[blocks.start:blocks.stop] = 1
    dist.all_reduce(owned)                                   # every block owned exactly once
    times = shard.max_over_ranks([10.0 + rank, 5.0 - rank])
    if rank == 0:
        out.put((owned.tolist(), times, list(blocks)))
    dist.barrier()
    dist.destroy_process_group()


def test_ranks_own_disjoint_blocks_and_reduce_max():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    owned, times, blocks0 = out.get(timeout=120)
    for p in procs:
        p.join(timeout=120)
        assert p.exitcode == 0
    assert owned == [1] * 56
    assert times == [11.0, 5.0]
    assert blocks0 == list(range(0, 32))                     # rank 0: 4 of the 7 streams


def test_stream_ranges_cover_without_overlap():
    sys.path.insert(0, ROOT)
    from paper_2605_02905_b200 import shard
    for streams in (0, 1, 5, 256):
        for world in (1, 2, 3, 8):
            seen = []
            for r in range(world):
                seen += list(shard.stream_range(streams, r, world))
            assert seen == list(range(streams))
