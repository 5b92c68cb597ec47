"""The allocation-free encode entry point against the ordinary one.

``eosq_encode_static`` is for callers that cannot call cudaMalloc where they compress (a serving
loop with a fixed memory plan, a plug-in without an allocator): its scratch is a fixed device array
inside the library.  It runs the same kernels as ``eosq_encode``, so through the C ABI its
output must agree with that entry point's -- here on two calls in a row with different blocks,
sizes and seeds, so that whatever the first call left in the shared array cannot leak into the
second.  This file sorts last on purpose: a run that stops at the first failure has then already
run every other test.
"""
import ctypes

import gc

import pytest
import torch

import paper_2605_02905_b200 as eosq
from paper_2605_02905_b200 import synth

pytestmark = pytest.mark.gpu

FIELDS = ("codes", "norms", "rank", "sigma", "phi", "V", "status", "eig", "lambda_plus")


def _same(a: eosq.Cache, b: eosq.Cache):
    # the same kernels on the same inputs: every array must be equal bit for bit
    for name in FIELDS:
        assert torch.equal(getattr(a, name), getattr(b, name)), name
    for blk in range(a.num_blocks):
        r = int(a.rank[blk])   # factor rows beyond the rank are not written
        assert torch.equal(a.P[blk, :r], b.P[blk, :r]), f"P of block {blk}"


def _device_bytes_in_use():
    free, total = torch.cuda.mem_get_info()
    return total - free


def test_static_scratch_encode_matches_workspace_encode_twice():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2605_02905_b200 import build
    build.build()
    ctx = eosq.Context()
    try:
        cap = eosq.eosq_encode_static_max_blocks()
        assert cap >= 8
        first = synth.kv_cache_blocks("static_a", layers=1, kv_heads=2, tokens=4 * 256, n=256, rank_hi=8, seed=71)
        second = synth.kv_cache_blocks("static_b", layers=1, kv_heads=1, tokens=3 * 1024, n=1024, rank_hi=10, seed=72)
        for w, bits, seed in ((first, 2, 1234), (second, 3, 99)):
            dev = w.blocks.cuda()
            B, n, d = dev.shape
            assert B <= cap
            ref = eosq.eosq_encode(ctx, dev, bits, seed)
            out = eosq.Cache.allocate(B, n, d, bits)
            for name in FIELDS + ("P",):
                getattr(out, name).fill_(0)
            eosq.eosq_encode_static(ctx, dev, bits, seed, out)   # first call of this shape: kernels load, the rotation is uploaded
            torch.cuda.synchronize()
            _same(out, ref)
            assert eosq.eosq_check_status(ctx, out) == 0
            # a repeated call must leave the device's memory exactly as it found it: neither the
            # caching allocator nor the driver may have been asked for a byte
            for name in FIELDS + ("P",):
                getattr(out, name).fill_(0)
            gc.collect()   # tensors that earlier tests left in reference cycles go now, not during the call
            torch.cuda.synchronize()
            alloc0, reserved0, used0 = torch.cuda.memory_allocated(), torch.cuda.memory_reserved(), _device_bytes_in_use()
            eosq.eosq_encode_static(ctx, dev, bits, seed, out)
            torch.cuda.synchronize()
            assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
            assert _device_bytes_in_use() == used0
            _same(out, ref)

        # beyond the fixed scratch: refused with a clear error, nothing written
        big = torch.zeros((cap + 1, 256, 128), dtype=torch.float16, device="cuda")
        out = eosq.Cache.allocate(cap + 1, 256, 128, 2)
        out.rank.fill_(-7)
        with pytest.raises(eosq.EosqError) as err:
            eosq.eosq_encode_static(ctx, big, 2, 1234, out)
        assert err.value.code == eosq.EOSQ_ERR_BUFFER_TOO_SMALL and "exceeds" in str(err.value)
        torch.cuda.synchronize()
        assert bool((out.rank == -7).all())
        # empty input is a no-op
        empty = torch.empty((0, 256, 128), dtype=torch.float16, device="cuda")
        eosq.eosq_encode_static(ctx, empty, 2, 1234, eosq.Cache.allocate(0, 256, 128, 2))
    finally:
        ctx.close()
