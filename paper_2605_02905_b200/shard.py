"""Host-side sharding of a KV cache over ranks (one process per GPU).

Every (layer, KV head, K|V, block) tile is compressed independently (Algorithm 3 works on one
block), so ranks own disjoint ranges of whole (layer, head) streams and there is no data-path
collective; only timings are reduced (max over ranks).
"""
from __future__ import annotations


def stream_range(num_streams: int, rank: int, world: int) -> range:
    """Contiguous range of (layer, head) streams owned by ``rank``: sizes differ by at most one."""
    if world < 1 or not (0 <= rank < world) or num_streams < 0:
        raise ValueError("bad rank / world / stream count")
    base, extra = divmod(num_streams, world)
    lo = rank * base + min(rank, extra)
    return range(lo, lo + base + (1 if rank < extra else 0))


def block_range(num_streams: int, blocks_per_stream: int, rank: int, world: int) -> range:
    """Blocks of a [stream][K|V][block] cache owned by ``rank`` (both K and V of its streams)."""
    r = stream_range(num_streams, rank, world)
    per = 2 * blocks_per_stream
    return range(r.start * per, r.stop * per)


def max_over_ranks(values, device=None):
    """Element-wise maximum of a list of floats over all ranks (identity without a process group)."""
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()
