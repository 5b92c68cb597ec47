"""GPU parity tests: the CUDA library, called through its C ABI, against the CPU oracle on the
same seeded blocks.  Sizes span several tiles and ragged tails; the full-size case is checked on
sampled blocks in the launch configuration the benchmark times."""
import ctypes
import json
import math

import numpy as np
import pytest
import torch

import oracle
import paper_2605_02905_b200 as eosq
from paper_2605_02905_b200 import synth

import parity

pytestmark = pytest.mark.gpu

SEED = 1234


@pytest.fixture(scope="module")
def ctx():
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    from paper_2605_02905_b200 import build
    build.build()
    c = eosq.Context()
    yield c
    c.close()


def _encode(ctx, blocks_cpu, bits, seed=SEED, full=True):
    """full: ask for the optional `eig` output, which makes the library resolve the whole spectrum;
    without it (the benchmark's configuration) it resolves only the eigenvalues Algorithm 2 reads."""
    dev = blocks_cpu.cuda()
    B, n, d = dev.shape
    out = eosq.Cache.allocate(B, n, d, bits, diagnostics=True if full else "staged")
    cache = eosq.eosq_encode(ctx, dev, bits, seed, out=out)
    torch.cuda.synchronize()
    return dev, cache


def _report(name, rep):
    print(f"\n[parity] {name}: " + json.dumps({k: (round(v, 9) if isinstance(v, float) else v) for k, v in rep.items()}))


def test_pr1_reference_block(ctx):
    """Config 0: one 256 x 128 fp32 block, b = 2, rotation seed 0; three spikes kept, the fourth rejected."""
    w = synth.pr1_block(0)
    dev, cache = _encode(ctx, w.blocks, 2, seed=0)
    rep, enc = parity.compare_encode(w.blocks, cache, 2, 0)
    _report("pr1", rep)
    assert int(cache.rank[0]) == 3 and rep["rank_mismatch"] == 0
    assert rep["e2e_mismatch_out_band"] == 0
    dec = eosq.eosq_decode(ctx, cache, 0)
    parity.compare_decode(cache, dec, 2, 0)


@pytest.mark.parametrize("full", [True, False])
@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_small_fp16_blocks_all_bit_widths(ctx, bits, full):
    w = synth.kv_cache_blocks("small", layers=1, kv_heads=2, tokens=768, n=256, rank_hi=8, seed=20 + bits)
    dev, cache = _encode(ctx, w.blocks, bits, full=full)
    rep, enc = parity.compare_encode(w.blocks, cache, bits, SEED)
    _report(f"small_b{bits}", rep)
    assert rep["e2e_out_band_fraction"] < 1e-4
    for out_dtype in (torch.float32, torch.float16):
        dec = eosq.eosq_decode(ctx, cache, SEED, out_dtype=out_dtype)
        parity.compare_decode(cache, dec, bits, SEED, tol=1e-4 if out_dtype == torch.float32 else 1e-3)


@pytest.mark.parametrize("full", [True, False])
def test_llama_shaped_blocks_n1024(ctx, full):
    """Config 1 prefix: keys and values of the first heads, n = 1024, spikes, coloured noise, outlier channels."""
    w = synth.llama_1layer(max_blocks=20)
    pick = [0, 1, 7, 8, 9, 15, 16, 19]  # K blocks 0..7, V blocks 8..15, next head's K 16..
    dev, cache = _encode(ctx, w.blocks, 2, full=full)
    rep, enc = parity.compare_encode(w.blocks, cache, 2, SEED, blocks_idx=pick)
    _report("llama_n1024", rep)
    assert rep["e2e_out_band_fraction"] < 1e-4
    dec = eosq.eosq_decode(ctx, cache, SEED)
    parity.compare_decode(cache, dec, 2, SEED, blocks_idx=pick[:4])


def test_scores_match_oracle(ctx):
    """Keys-only view of a [head][K|V][block] cache: G = 4 query heads per KV head, and a wide group."""
    w = synth.kv_cache_blocks("scores", layers=1, kv_heads=3, tokens=512, n=256, rank_hi=6, seed=31)
    heads, bph = 3, 2
    for bits, G in ((2, 4), (3, 4), (4, 11), (1, 1)):
        dev, cache = _encode(ctx, w.blocks, bits)
        q = synth.queries(heads, G, seed=5).cuda()
        scale = 1.0 / math.sqrt(128)
        s = eosq.eosq_scores(ctx, cache, q, heads, bph, 2 * bph, SEED, scale)
        torch.cuda.synchronize()
        worst = parity.compare_scores(cache, q, s, heads, bph, 2 * bph, bits, SEED, scale)
        print(f"\n[parity] scores b={bits} G={G}: worst relative {worst:.3e}")


def test_degenerate_blocks(ctx):
    """Pure noise (rank 0), an all-zero block, a block with zero rows, a rank-one block."""
    g = torch.Generator().manual_seed(3)
    n, d = 256, 128
    noise = torch.randn(n, d, generator=g) * 0.3
    zero = torch.zeros(n, d)
    holes = torch.randn(n, d, generator=g) * 0.3
    holes[5] = 0
    holes[200:210] = 0
    rank1 = torch.randn(n, 1, generator=g) @ torch.randn(1, d, generator=g) + 0.05 * torch.randn(n, d, generator=g)
    blocks = torch.stack([noise, zero, holes, rank1]).to(torch.float16)
    dev, fast = _encode(ctx, blocks, 2, full=False)
    rep, enc = parity.compare_encode(blocks, fast, 2, SEED)
    _report("degenerate_top_eigenvalues_only", rep)
    dev, cache = _encode(ctx, blocks, 2)
    assert torch.equal(fast.rank, cache.rank) and torch.equal(fast.status, cache.status)
    rep, enc = parity.compare_encode(blocks, cache, 2, SEED, enc=enc)
    _report("degenerate", rep)
    ranks = cache.rank.cpu().tolist()
    assert ranks[0] == 0 and ranks[1] == 0 and ranks[2] == 0 and ranks[3] == 1
    norms = cache.norms.cpu()
    assert torch.all(norms[1] == 0) and norms[2][5] == 0 and torch.all(norms[2][200:210] == 0)
    dec = eosq.eosq_decode(ctx, cache, SEED)
    assert torch.all(dec[1] == 0) and torch.all(dec[2][5] == 0)
    parity.compare_decode(cache, dec, 2, SEED)


@pytest.mark.parametrize("full", [True, False])
@pytest.mark.parametrize("n", [128, 136, 4096])
def test_ragged_and_extreme_block_lengths(ctx, n, full):
    """n = d (square), n not a multiple of the row tile, and the largest supported n."""
    w = synth.kv_cache_blocks("ragged", layers=1, kv_heads=1, tokens=2 * n, n=n, rank_hi=5, seed=40 + n)
    dev, cache = _encode(ctx, w.blocks, 3, full=full)
    rep, enc = parity.compare_encode(w.blocks, cache, 3, SEED, blocks_idx=[0, 3] if n == 4096 else None)
    _report(f"n{n}", rep)
    dec = eosq.eosq_decode(ctx, cache, SEED)
    parity.compare_decode(cache, dec, 3, SEED, blocks_idx=[0] if n == 4096 else None)
    q = synth.queries(2, 4, seed=6).cuda()
    s = eosq.eosq_scores(ctx, cache, q, 2, 2, 2, SEED)
    parity.compare_scores(cache, q, s, 2, 2, 2, 3, SEED, 1.0 / math.sqrt(128), pairs=[(0, 0), (1, 1)])


@pytest.mark.parametrize("n", [136, 1000])
def test_two_bit_decode_with_a_ragged_last_tile(ctx, n):
    """The tensor-core decode (2-bit codes) on blocks whose length is not a multiple of its 128-token tile,
    an odd number of blocks (the two halves of its CTA get different counts), both output types."""
    w = synth.kv_cache_blocks("ragged2", layers=1, kv_heads=1, tokens=n, n=n, rank_hi=6, seed=70 + n)
    blocks = torch.cat([w.blocks, w.blocks[:1] * 0.5], dim=0)   # 3 blocks
    dev, cache = _encode(ctx, blocks, 2)
    for out_dtype in (torch.float16, torch.float32):
        dec = eosq.eosq_decode(ctx, cache, SEED, out_dtype=out_dtype)
        parity.compare_decode(cache, dec, 2, SEED, tol=1e-4 if out_dtype == torch.float32 else 1e-3)
    assert eosq.eosq_check_status(ctx, cache) == 0


def test_many_blocks_cross_the_chunk_boundary_and_are_deterministic(ctx):
    """More blocks than one internal chunk (18944): every block must equal its stand-alone encoding."""
    w = synth.kv_cache_blocks("chunks", layers=2, kv_heads=3, tokens=128 * 1580, n=128, rank_hi=4, seed=50, device="cuda")
    B = w.blocks.shape[0]
    assert B == 18960
    cache = eosq.eosq_encode(ctx, w.blocks, 2, SEED)
    cache2 = eosq.eosq_encode(ctx, w.blocks, 2, SEED)
    torch.cuda.synchronize()
    for name in ("codes", "norms", "rank", "sigma", "phi", "V", "status", "eig"):
        assert torch.equal(getattr(cache, name), getattr(cache2, name)), name
    del cache2
    pick = [0, 591, 18943, 18944, B - 1]
    for b in pick:
        single = eosq.eosq_encode(ctx, w.blocks[b:b + 1].contiguous(), 2, SEED)
        assert torch.equal(single.codes[0], cache.codes[b]) and torch.equal(single.norms[0], cache.norms[b])
        r = int(single.rank[0])
        assert r == int(cache.rank[b]) and torch.equal(single.P[0, :r], cache.P[b, :r])
    sub = w.blocks[pick].cpu()
    sub_cache = eosq.Cache.allocate(len(pick), w.n, w.d, 2)
    for name in ("codes", "norms", "rank", "sigma", "phi", "P", "V", "status", "eig", "lambda_plus", "vr32", "coef"):
        getattr(sub_cache, name).copy_(getattr(cache, name)[pick])
    rep, enc = parity.compare_encode(sub, sub_cache, 2, SEED)
    _report("chunks", rep)


def test_profile_select_times_only_the_chosen_stage(ctx):
    """eosq_profile_select brackets the launches of the named stages only; the count of all launches goes on."""
    w = synth.kv_cache_blocks("prof", layers=1, kv_heads=2, tokens=512, n=256, rank_hi=4, seed=61)
    n0 = ctx.launch_count
    ctx.profile_select(["quant", "tridiag_b"])
    try:
        _encode(ctx, w.blocks, 2)
        stages = ctx.profile_read()
    finally:
        ctx.profile_enable(False)
    timed = {k for k, v in stages.items() if v[1]}
    assert timed == {"quant", "tridiag_b"}, timed
    assert stages["quant"][0] > 0.0 and stages["quant"][1] == 1
    assert ctx.launch_count - n0 >= 6   # Gram, tridiagonalisation ranges, eigenvalues, spectral, quantise (and the second pass)


def test_host_buffer_entry_point_matches_device_path(ctx):
    w = synth.kv_cache_blocks("host", layers=1, kv_heads=2, tokens=512, n=256, rank_hi=6, seed=60)
    dev, cache = _encode(ctx, w.blocks, 2)
    B, n, d = w.blocks.shape
    host_in = w.blocks.pin_memory()
    host_out = eosq.Cache.allocate(B, n, d, 2, pinned=True, diagnostics=False)
    host_out.eig = torch.empty((B, d), dtype=torch.float32).pin_memory()
    arena = torch.empty(eosq.eosq_encode_host_arena_bytes(B, n, d, 2, eosq.EOSQ_F16), dtype=torch.uint8, device="cuda")
    eosq.eosq_encode_host(ctx, host_in, 2, SEED, host_out, arena)
    for name in ("codes", "norms", "rank", "sigma", "phi", "V", "status", "eig"):
        assert torch.equal(getattr(host_out, name), getattr(cache, name).cpu()), name
    for b in range(B):
        r = int(cache.rank[b])
        assert torch.equal(host_out.P[b, :r], cache.P[b, :r].cpu())


def test_empty_input_and_argument_errors(ctx):
    L = eosq.lib()
    empty = torch.empty((0, 256, 128), dtype=torch.float16, device="cuda")
    cache = eosq.eosq_encode(ctx, empty, 2, SEED)
    assert cache.num_blocks == 0
    assert eosq.eosq_decode(ctx, cache, SEED).shape == (0, 256, 128)
    blocks = torch.zeros((2, 256, 128), dtype=torch.float16, device="cuda")
    good = eosq.Cache.allocate(2, 256, 128, 2)
    st = good.struct()
    ws = torch.empty(eosq.eosq_workspace_bytes(2, 256, 128), dtype=torch.uint8, device="cuda")
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def call(blocks_ptr=blocks.data_ptr(), dtype=eosq.EOSQ_F16, B=2, n=256, d=128, bits=2, out=ctypes.addressof(st),
             wsp=ws.data_ptr(), wsb=ws.numel()):
        return L.eosq_encode(ctx._h, blocks_ptr, dtype, B, n, d, bits, ctypes.c_uint64(SEED), out, wsp, wsb, stream)

    assert call() == eosq.EOSQ_OK
    assert call(blocks_ptr=None) == eosq.EOSQ_ERR_INVALID_ARG
    assert call(out=None) == eosq.EOSQ_ERR_INVALID_ARG
    assert call(dtype=7) == eosq.EOSQ_ERR_INVALID_ARG
    assert call(B=-1) == eosq.EOSQ_ERR_INVALID_ARG
    assert call(blocks_ptr=blocks.data_ptr() + 2) == eosq.EOSQ_ERR_INVALID_ARG
    assert call(d=64) == eosq.EOSQ_ERR_UNSUPPORTED
    assert call(bits=5) == eosq.EOSQ_ERR_UNSUPPORTED
    assert call(n=64) == eosq.EOSQ_ERR_UNSUPPORTED
    assert call(n=8192) == eosq.EOSQ_ERR_UNSUPPORTED
    assert call(wsb=1024) == eosq.EOSQ_ERR_BUFFER_TOO_SMALL
    missing = eosq.Cache.allocate(2, 256, 128, 2)
    missing.norms = None
    st2 = missing.struct()
    assert call(out=ctypes.addressof(st2)) == eosq.EOSQ_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert eosq.eosq_check_status(ctx, good) == 0


def test_nonfinite_input_is_flagged_not_fatal(ctx):
    blocks = torch.randn(2, 256, 128, generator=torch.Generator().manual_seed(1)).to(torch.float16)
    blocks[1, 3, 7] = float("inf")
    dev, cache = _encode(ctx, blocks, 2)
    status = cache.status.cpu().tolist()
    assert status[0] == 0 and status[1] != 0
    assert eosq.eosq_check_status(ctx, cache) == 1


@pytest.mark.parametrize("bits,full", [(2, False), (3, True)])
def test_full_size_cache_sampled_blocks(ctx, bits, full):
    """Config 2 in the benchmark's launch configuration (both of its code widths): the whole
    Llama-3.1-8B-shaped 32k cache (16384 blocks, 4 GiB) is encoded, scored and decoded in one call each;
    sampled blocks go to the oracle one by one, and properties that hold at any size are checked on everything.
    b = 2 runs as the benchmark does (only the eigenvalues Algorithm 2 reads), b = 3 with the whole spectrum."""
    w = synth.llama_32k(device="cuda")
    B = w.blocks.shape[0]
    assert B == 16384
    cache = eosq.Cache.allocate(B, w.n, w.d, bits, diagnostics=True if full else "staged")
    eosq.eosq_encode(ctx, w.blocks, bits, SEED, out=cache)
    torch.cuda.synchronize()
    assert eosq.eosq_check_status(ctx, cache) == 0
    ranks = cache.rank
    assert int(ranks.min()) >= 0 and int(ranks.max()) <= 11
    assert torch.all(torch.isfinite(cache.norms.float()))
    if full:
        eig = cache.eig
        assert torch.all(eig[:, :-1] >= eig[:, 1:]) and torch.all(eig[:, -1] > -1e-3 * eig[:, 0])
        # Frobenius identity: sum of eigenvalues of the Gram matrix = ||S||_F^2
        fro = (w.blocks[:256].float() ** 2).sum(dim=(1, 2))
        assert torch.allclose(eig[:256].sum(dim=1), fro, rtol=2e-3)
    pick = [0, 31, 32, 4097, 9000, B - 1]
    sub = w.blocks[pick].cpu()
    sub_cache = eosq.Cache.allocate(len(pick), w.n, w.d, bits, diagnostics=True if full else "staged")
    for name in ("codes", "norms", "rank", "sigma", "phi", "P", "V", "status", "eig", "lambda_plus", "vr32", "coef"):
        if getattr(cache, name) is not None:
            getattr(sub_cache, name).copy_(getattr(cache, name)[pick])
    rep, enc = parity.compare_encode(sub, sub_cache, bits, SEED)
    _report(f"llama_32k_sampled_b{bits}", rep)
    assert rep["e2e_out_band_fraction"] < 1e-4
    # scores over the keys of the first layers, sampled (head, block) pairs against the oracle
    heads, bph, G = 16, 32, 4
    q = synth.queries(heads, G, seed=8).cuda()
    s = eosq.eosq_scores(ctx, cache, q, heads, bph, 2 * bph, SEED)
    torch.cuda.synchronize()
    parity.compare_scores(cache, q, s, heads, bph, 2 * bph, bits, SEED, 1.0 / math.sqrt(128), pairs=[(0, 0), (5, 17), (15, 31)])
    # decode of the whole cache to fp16; the sampled blocks against the oracle's decode of the same stored bytes
    del s
    dec = eosq.eosq_decode(ctx, cache, SEED, out_dtype=torch.float16)
    torch.cuda.synchronize()
    assert eosq.eosq_check_status(ctx, cache) == 0
    assert torch.all(torch.isfinite(dec[::257].float()))
    parity.compare_decode(sub_cache, dec[pick], bits, SEED, tol=1e-3)


def test_full_size_ministral_cache_sampled_blocks(ctx):
    """Config 3 at its full size and in the benchmark's launch configuration: the Ministral-8B-shaped 64k
    cache (36864 blocks, 9 GiB; two chunks of the library's scratch) is encoded at b = 2 in one call, the
    logits of G = 16 queries per KV head (4 query heads x batch 4) are taken against compressed keys, and
    blocks sampled on both sides of the chunk boundary go to the oracle one by one."""
    w = synth.ministral_64k(device="cuda")
    B = w.blocks.shape[0]
    assert B == 36864
    cache = eosq.Cache.allocate(B, w.n, w.d, 2, diagnostics="staged")
    eosq.eosq_encode(ctx, w.blocks, 2, SEED, out=cache)
    torch.cuda.synchronize()
    assert eosq.eosq_check_status(ctx, cache) == 0
    ranks = cache.rank
    assert int(ranks.min()) >= 0 and int(ranks.max()) <= 11
    assert torch.all(torch.isfinite(cache.norms.float()))
    planted = w.planted_rank
    noise_values = [i for i in range(B) if planted[i] == 0 and not bool(w.is_key[i])]
    assert noise_values and all(int(ranks[i]) == 0 for i in noise_values[:200])
    pick = sorted({0, 63, 64, 18943, 18944, 18945, 30001, B - 1, noise_values[0]})
    sub = w.blocks[pick].cpu()
    sub_cache = eosq.Cache.allocate(len(pick), w.n, w.d, 2, diagnostics="staged")
    for name in ("codes", "norms", "rank", "sigma", "phi", "P", "V", "status", "lambda_plus", "vr32", "coef"):
        getattr(sub_cache, name).copy_(getattr(cache, name)[pick])
    rep, enc = parity.compare_encode(sub, sub_cache, 2, SEED)
    _report("ministral_64k_sampled_b2", rep)
    assert rep["e2e_out_band_fraction"] < 1e-4
    heads, bph, G = 8, 64, 16
    q = synth.queries(heads, G, seed=9).cuda()
    s = eosq.eosq_scores(ctx, cache, q, heads, bph, 2 * bph, SEED)
    torch.cuda.synchronize()
    assert eosq.eosq_check_status(ctx, cache) == 0
    parity.compare_scores(cache, q, s, heads, bph, 2 * bph, 2, SEED, 1.0 / math.sqrt(128), pairs=[(0, 0), (3, 40), (7, 63)])


def _stratified(planted, is_key, want):
    """Indices of blocks covering the planted ranks in `want` for keys and values (first match each)."""
    pick = []
    for key in (True, False):
        for lo, hi in want:
            hits = [i for i in range(len(planted)) if bool(is_key[i]) == key and lo <= planted[i] <= hi and i not in pick]
            if hits:
                pick.append(hits[0])
    return sorted(pick)


def test_ministral_shaped_blocks_rank_above_pilot_and_pure_noise(ctx):
    """Config 3 (Ministral-8B shape, n = 1024): planted ranks up to 32, above the pilot k = 11, where the
    single-pass rank test of Algorithm 2 inflates its own bulk edge and the selected rank collapses; 5 % of
    the blocks are pure noise (rank 0).  Keys and values, sampled by planted rank; then the logits of
    G = 16 queries per KV head (4 query heads x batch 4) against the compressed keys of the first head."""
    w = synth.ministral_64k(max_blocks=136)            # head 0: K blocks 0..63, V blocks 64..127, then head 1's K
    planted = w.planted_rank
    pick = _stratified(planted, w.is_key, [(0, 0), (1, 4), (5, 11), (12, 20), (21, 32)])
    assert any(planted[i] == 0 for i in pick) and any(planted[i] > 11 for i in pick)
    dev, cache = _encode(ctx, w.blocks, 2, full=False)
    flagged = {i: int(v) for i, v in enumerate(cache.status.cpu().tolist()) if v}
    assert not flagged, flagged
    rep, enc = parity.compare_encode(w.blocks, cache, 2, SEED, blocks_idx=pick)
    rep["planted_vs_selected"] = [(int(planted[i]), int(cache.rank[i])) for i in pick]
    _report("ministral_n1024", rep)
    assert rep["e2e_out_band_fraction"] < 1e-4
    sel = cache.rank.cpu().numpy()
    # pure-noise value blocks must come out with rank 0 (key blocks still carry their outlier channels)
    assert sel.max() <= 11 and all(sel[i] == 0 for i in range(len(planted)) if planted[i] == 0 and not w.is_key[i])
    dec = eosq.eosq_decode(ctx, cache, SEED)
    parity.compare_decode(cache, dec, 2, SEED, blocks_idx=pick[:3])
    heads, bph, G = 1, 64, 16
    q = synth.queries(heads, G, seed=12).cuda()
    s = eosq.eosq_scores(ctx, cache, q, heads, bph, 2 * bph, SEED)
    torch.cuda.synchronize()
    worst = parity.compare_scores(cache, q, s, heads, bph, 2 * bph, 2, SEED, 1.0 / math.sqrt(128),
                                  pairs=[(0, 0), (0, 17), (0, 63)])
    print(f"\n[parity] ministral scores G=16: worst relative {worst:.3e}")


@pytest.mark.parametrize("n", [256, 512, 1024, 2048, 4096])
def test_sweep_points_around_the_detection_threshold(ctx, n):
    """Config 4 (sweep): four spikes at {5, 1.5, 1.05, 0.9} x the BBP threshold, block lengths 256 .. 4096, every
    code width.  The 0.9 x and 1.05 x spikes sit at the bulk edge and must not be kept; the 1.5 x one lands
    close to the d^(-1/3) margin of the rank test."""
    w = synth.kv_cache_blocks(f"sweep_n{n}", layers=1, kv_heads=1, tokens=3 * n, n=n, fixed_theta=[5.0, 1.5, 1.05, 0.9], seed=4)
    pick = [0, 4] if n >= 2048 else [0, 2, 4]          # K blocks 0..2, V blocks 3..5
    enc2 = None
    hist = {}
    for bits in (2, 1, 3, 4):
        dev, cache = _encode(ctx, w.blocks, bits, full=(bits == 3))
        rep, enc = parity.compare_encode(w.blocks, cache, bits, SEED, blocks_idx=pick)
        if bits == 2:
            enc2 = enc
            for r in cache.rank.cpu().tolist():
                hist[r] = hist.get(r, 0) + 1
            rep["rank_histogram"] = hist
            rep["min_margin"] = float(enc["margin"].min())
        _report(f"sweep_n{n}_b{bits}", rep)
        assert rep["e2e_out_band_fraction"] < 1e-4
        # value blocks: the 5 x spike always kept, the 1.5 x one at most, the edge spikes never; key blocks
        # add their four outlier channels
        sel = cache.rank.cpu().numpy()
        assert all(1 <= sel[i] <= 2 for i in range(len(sel)) if not w.is_key[i]), sel
        assert all(1 <= sel[i] <= 6 for i in range(len(sel)) if w.is_key[i]), sel
    dec = eosq.eosq_decode(ctx, cache, SEED)
    parity.compare_decode(cache, dec, 4, SEED, blocks_idx=pick[:1])
    assert enc2 is not None


def test_block_at_the_rank_threshold_is_compared_separately(ctx):
    """A block whose leading eigenvalue sits within 1e-4 of the rank cut (strength found by bisection on the
    oracle): either side of the cut is a valid answer there, so the comparison must take its
    near-threshold branch -- same rank and full parity, or a flagged mismatch -- and count the block."""
    n, d = 256, 128
    g = torch.Generator().manual_seed(11)
    Z = torch.randn(n, d, generator=g, dtype=torch.float64) / math.sqrt(n)
    u = torch.linalg.qr(torch.randn(n, 1, generator=g, dtype=torch.float64))[0]
    v = torch.linalg.qr(torch.randn(d, 1, generator=g, dtype=torch.float64))[0]

    def block(theta):
        return ((Z + theta * (u @ v.T)) * 4.0).to(torch.float16)

    def state(theta):
        S = block(theta).double().numpy()
        sig = oracle.svd(S)[0]
        sp = oracle.eoptshrink_spectrum(n, d, sig)
        return sp["rank"], sp["margin"]

    lo, hi = 0.5, 3.0
    assert state(lo)[0] == 0 and state(hi)[0] == 1
    theta = hi
    for _ in range(60):
        mid = 0.5 * (lo + hi)
        r, margin = state(mid)
        theta = mid
        if margin < 5e-5:
            break
        if r == 0:
            lo = mid
        else:
            hi = mid
    r, margin = state(theta)
    assert margin < parity.RANK_MARGIN, margin
    blocks = torch.stack([block(theta), block(theta * 1.5)])
    dev, cache = _encode(ctx, blocks, 2, full=False)
    rep, enc = parity.compare_encode(blocks, cache, 2, SEED)
    rep["margin"] = margin
    _report("near_threshold", rep)
    assert rep["near_threshold_blocks"] == 1
    assert int(cache.rank[1]) == 1 and int(cache.rank[0]) in (0, 1)


def test_unaligned_cache_arrays_are_rejected(ctx):
    """Decode and scores move the cache with 16-byte bulk copies: a misaligned array is an argument error."""
    L = eosq.lib()
    blocks = torch.randn(2, 256, 128, generator=torch.Generator().manual_seed(2)).to(torch.float16)
    dev, cache = _encode(ctx, blocks, 2)
    st = cache.struct()
    st.codes = cache.codes.data_ptr() + 4
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    out = torch.empty((2, 256, 128), dtype=torch.float32, device="cuda")
    rc = L.eosq_decode(ctx._h, ctypes.addressof(st), 2, 256, 128, 2, ctypes.c_uint64(SEED), out.data_ptr(), eosq.EOSQ_F32, stream)
    assert rc == eosq.EOSQ_ERR_INVALID_ARG
    q = synth.queries(1, 4, seed=1).cuda()
    s = torch.empty((1, 4, 512), dtype=torch.float32, device="cuda")
    rc = L.eosq_scores(ctx._h, ctypes.addressof(st), 1, 2, 2, 256, 128, 2, ctypes.c_uint64(SEED), q.data_ptr(), 4,
                       ctypes.c_float(0.1), s.data_ptr(), stream)
    assert rc == eosq.EOSQ_ERR_INVALID_ARG


def test_a_wait_that_runs_out_is_reported_once_and_the_context_stays_usable(ctx):
    """The time-out path without a hang: a kernel waits (a few hundred microseconds at most) on a barrier
    nothing arrives at, gives up, and the context reports it as an error of the next status check; after
    that the same context compresses as before."""
    w = synth.kv_cache_blocks("timeout", layers=1, kv_heads=2, tokens=512, n=256, rank_hi=4, seed=77)
    blocks = w.blocks.cuda()
    before = eosq.eosq_encode(ctx, blocks, 2, SEED)
    assert eosq.eosq_check_status(ctx, before) == 0
    L = eosq.lib()
    assert L.eosq_selftest_wait_timeout(ctx._h, 0, None) == eosq.EOSQ_ERR_INVALID_ARG
    assert L.eosq_selftest_wait_timeout(ctx._h, 5000, None) == eosq.EOSQ_ERR_INVALID_ARG
    ctx.selftest_wait_timeout(polls=128)
    with pytest.raises(eosq.EosqError) as err:
        eosq.eosq_check_status(ctx, before)
    assert err.value.code == eosq.EOSQ_ERR_CUDA and "kernel bits 32" in str(err.value)
    assert eosq.eosq_check_status(ctx, before) == 0          # reported once
    after = eosq.eosq_encode(ctx, blocks, 2, SEED)
    assert eosq.eosq_check_status(ctx, after) == 0
    for name in ("codes", "norms", "rank", "sigma", "phi", "V", "status"):
        assert torch.equal(getattr(before, name), getattr(after, name)), name
