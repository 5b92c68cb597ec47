"""Python binding of the eosq C-ABI library (argument marshalling only).

Every step of the compression path runs inside ``libeosq.so`` (hand-written CUDA for
sm_100a); PyTorch is used here for device memory and streams.  The functions carry the
names of the C entry points declared in ``include/eosq.h``.  There is no CPU fallback:
if the library has not been built the first call raises.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
from pathlib import Path
from typing import Optional

import numpy as np

_PKG = Path(__file__).resolve().parent
LIB_PATH = _PKG / "libeosq.so"

EOSQ_OK, EOSQ_ERR_INVALID_ARG, EOSQ_ERR_UNSUPPORTED, EOSQ_ERR_BUFFER_TOO_SMALL, EOSQ_ERR_CUDA, EOSQ_WARN_BLOCK_STATUS = range(6)
EOSQ_F16, EOSQ_F32 = 0, 1
EOSQ_RMAX = 16
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "BUFFER_TOO_SMALL", 4: "CUDA", 5: "BLOCK_STATUS"}

EXPORTS = [
    "eosq_pilot_k", "eosq_codebook", "eosq_rotation", "eosq_layout", "eosq_bits_per_entry",
    "eosq_workspace_bytes", "eosq_create", "eosq_destroy", "eosq_last_cuda_error", "eosq_encode",
    "eosq_decode", "eosq_scores", "eosq_encode_host_arena_bytes", "eosq_encode_host",
    "eosq_check_status", "eosq_launch_count", "eosq_profile_enable", "eosq_profile_select", "eosq_profile_read",
    "eosq_encode_static", "eosq_encode_static_max_blocks", "eosq_selftest_wait_timeout",
]
STAGES = ["gram", "tridiag_a", "tridiag_b", "tridiag_c", "eigvals", "spectral", "quant", "decode", "scores", "redo", "other"]


class EosqError(RuntimeError):
    def __init__(self, code, what, detail=""):
        super().__init__(f"{what}: EOSQ_{STATUS_NAMES.get(code, code)}" + (f" ({detail})" if detail else ""))
        self.code = code


class _CacheStruct(ctypes.Structure):
    _fields_ = [(name, ctypes.c_void_p) for name in
                ("codes", "norms", "rank", "sigma", "phi", "P", "V", "status", "eig", "lambda_plus", "vr32", "coef")]


class _LayoutStruct(ctypes.Structure):
    _fields_ = [("k", ctypes.c_int32), ("rmax", ctypes.c_int32), ("row_bytes", ctypes.c_int32),
                ("reserved", ctypes.c_int32)] + [
        (name, ctypes.c_int64) for name in
        ("codes_bytes", "norms_bytes", "P_bytes", "V_bytes", "sigma_bytes", "phi_bytes", "eig_bytes", "stored_bytes")]


_lib = None


def lib():
    """The loaded shared library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not LIB_PATH.exists():
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2605_02905_b200.build` "
                "(nvcc, sm_100a).  There is no CPU fallback.")
        L = ctypes.CDLL(str(LIB_PATH))
        L.eosq_bits_per_entry.restype = ctypes.c_double
        L.eosq_bits_per_entry.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_int]
        L.eosq_workspace_bytes.restype = ctypes.c_size_t
        L.eosq_workspace_bytes.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.c_int]
        L.eosq_encode_host_arena_bytes.restype = ctypes.c_size_t
        L.eosq_encode_host_arena_bytes.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int]
        L.eosq_last_cuda_error.restype = ctypes.c_char_p
        L.eosq_last_cuda_error.argtypes = [ctypes.c_void_p]
        L.eosq_launch_count.restype = ctypes.c_int64
        L.eosq_launch_count.argtypes = [ctypes.c_void_p]
        L.eosq_rotation.argtypes = [ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p]
        L.eosq_codebook.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p]
        L.eosq_layout.argtypes = [ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_void_p]
        L.eosq_create.argtypes = [ctypes.c_void_p]
        L.eosq_destroy.argtypes = [ctypes.c_void_p]
        L.eosq_encode.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                  ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.eosq_encode_static.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                         ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p]
        L.eosq_encode_static_max_blocks.restype = ctypes.c_int64
        L.eosq_encode_static_max_blocks.argtypes = []
        L.eosq_decode.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                  ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p]
        L.eosq_scores.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ctypes.c_int,
                                  ctypes.c_int, ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_int, ctypes.c_float,
                                  ctypes.c_void_p, ctypes.c_void_p]
        L.eosq_encode_host.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_int, ctypes.c_int,
                                       ctypes.c_int, ctypes.c_uint64, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        L.eosq_selftest_wait_timeout.argtypes = [ctypes.c_void_p, ctypes.c_uint32, ctypes.c_void_p]
        L.eosq_profile_enable.argtypes = [ctypes.c_void_p, ctypes.c_int]
        L.eosq_profile_select.argtypes = [ctypes.c_void_p, ctypes.c_uint32]
        L.eosq_profile_read.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
        L.eosq_check_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
        _lib = L
    return _lib


def _check(rc, what, ctx=None):
    if rc != EOSQ_OK:
        detail = ""
        if rc == EOSQ_ERR_CUDA and ctx is not None:
            detail = lib().eosq_last_cuda_error(ctx._h).decode()
        raise EosqError(rc, what, detail)


# ---- host-side pure functions ------------------------------------------------------------

def eosq_pilot_k(d: int) -> int:
    return int(lib().eosq_pilot_k(int(d)))


def eosq_codebook(bits: int, d: int):
    cen = np.zeros(1 << bits, dtype=np.float64)
    thr = np.zeros((1 << bits) - 1, dtype=np.float64)
    _check(lib().eosq_codebook(int(bits), int(d), cen.ctypes.data, thr.ctypes.data), "eosq_codebook")
    return cen, thr


def eosq_rotation(d: int, seed: int):
    pi = np.zeros((d, d), dtype=np.float64)
    _check(lib().eosq_rotation(int(d), ctypes.c_uint64(seed), pi.ctypes.data), "eosq_rotation")
    return pi


def eosq_layout(n: int, d: int, bits: int) -> dict:
    s = _LayoutStruct()
    _check(lib().eosq_layout(int(n), int(d), int(bits), ctypes.addressof(s)), "eosq_layout")
    return {name: int(getattr(s, name)) for name, _ in _LayoutStruct._fields_ if name != "reserved"}


def eosq_bits_per_entry(bits: int, rank: float, n: int, d: int, b_s: float, prod: bool = False) -> float:
    return float(lib().eosq_bits_per_entry(int(bits), float(rank), int(n), int(d), float(b_s), int(bool(prod))))


def eosq_workspace_bytes(num_blocks: int, n: int, d: int) -> int:
    return int(lib().eosq_workspace_bytes(int(num_blocks), int(n), int(d)))


def eosq_encode_host_arena_bytes(num_blocks: int, n: int, d: int, bits: int, in_dtype: int) -> int:
    return int(lib().eosq_encode_host_arena_bytes(int(num_blocks), int(n), int(d), int(bits), int(in_dtype)))


# ---- context and compressed cache ----------------------------------------------------------

class Context:
    """Owner of an ``eosq_ctx`` on the current CUDA device."""

    def __init__(self):
        h = ctypes.c_void_p()
        _check(lib().eosq_create(ctypes.byref(h)), "eosq_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            lib().eosq_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def selftest_wait_timeout(self, polls: int = 64, stream=None):
        """Launches the kernel whose bounded wait runs out; the next check_status reports it."""
        _check(lib().eosq_selftest_wait_timeout(self._h, int(polls), _stream_ptr(stream)), "eosq_selftest_wait_timeout", self)

    @property
    def launch_count(self) -> int:
        return int(lib().eosq_launch_count(self._h))

    def profile_enable(self, on: bool = True):
        _check(lib().eosq_profile_enable(self._h, int(bool(on))), "eosq_profile_enable", self)

    def profile_select(self, stages):
        """Times only the named stages (see STAGES)."""
        mask = 0
        for name in stages:
            mask |= 1 << STAGES.index(name)
        _check(lib().eosq_profile_select(self._h, mask), "eosq_profile_select", self)

    def profile_read(self) -> dict:
        """{stage: (milliseconds, launches)} accumulated since the last read (synchronises)."""
        ms = (ctypes.c_float * len(STAGES))()
        cnt = (ctypes.c_int64 * len(STAGES))()
        _check(lib().eosq_profile_read(self._h, ms, cnt), "eosq_profile_read", self)
        return {STAGES[i]: (float(ms[i]), int(cnt[i])) for i in range(len(STAGES))}


@dataclass
class Cache:
    """Structure-of-arrays compressed cache (``eosq_cache_t``) held in torch tensors."""
    num_blocks: int
    n: int
    d: int
    bits: int
    codes: "object"
    norms: "object"
    rank: "object"
    sigma: "object"
    phi: "object"
    P: "object"
    V: "object"
    status: "object"
    eig: Optional["object"] = None
    lambda_plus: Optional["object"] = None
    vr32: Optional["object"] = None
    coef: Optional["object"] = None

    @staticmethod
    def allocate(num_blocks, n, d, bits, device="cuda", diagnostics=True, pinned=False):
        import torch
        kw = dict(device=device) if not pinned else dict(device="cpu", pin_memory=True)
        B = max(int(num_blocks), 0)
        c = Cache(
            B, n, d, bits,
            codes=torch.empty((B, n, d * bits // 8), dtype=torch.uint8, **kw),
            norms=torch.empty((B, n), dtype=torch.float16, **kw),
            rank=torch.empty((B,), dtype=torch.int32, **kw),
            sigma=torch.empty((B, EOSQ_RMAX), dtype=torch.float32, **kw),
            phi=torch.empty((B, EOSQ_RMAX), dtype=torch.float32, **kw),
            P=torch.empty((B, EOSQ_RMAX, n), dtype=torch.float16, **kw),
            V=torch.empty((B, EOSQ_RMAX, d), dtype=torch.float16, **kw),
            status=torch.empty((B,), dtype=torch.int32, **kw),
        )
        # diagnostics: True = every optional array; "staged" = all but the full spectrum `eig`
        # (asking for `eig` makes eosq_encode resolve all d eigenvalues instead of the 3k + 2 it needs)
        if diagnostics and diagnostics != "staged":
            c.eig = torch.empty((B, d), dtype=torch.float32, **kw)
        if diagnostics:
            c.lambda_plus = torch.empty((B,), dtype=torch.float32, **kw)
            c.vr32 = torch.empty((B, EOSQ_RMAX, d), dtype=torch.float32, **kw)
            c.coef = torch.empty((B, EOSQ_RMAX), dtype=torch.float32, **kw)
        return c

    def struct(self) -> _CacheStruct:
        s = _CacheStruct()
        for name, _ in _CacheStruct._fields_:
            t = getattr(self, name)
            setattr(s, name, t.data_ptr() if t is not None and t.numel() > 0 else None)
        return s

    def stored_bytes(self) -> int:
        """Bytes eosq_scores / eosq_decode read per pass: codes, norms and the kept factor rows."""
        r = int(self.rank.sum().item())
        return int(self.codes.numel() + 2 * self.norms.numel() + 2 * r * (self.n + self.d))


def _stream_ptr(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return ctypes.c_void_p(s.cuda_stream)


def _dtype_code(t):
    import torch
    if t.dtype == torch.float16:
        return EOSQ_F16
    if t.dtype == torch.float32:
        return EOSQ_F32
    raise TypeError(f"blocks must be float16 or float32, got {t.dtype}")


def eosq_encode(ctx: Context, blocks, bits: int, seed: int, out: Optional[Cache] = None, workspace=None, stream=None) -> Cache:
    """blocks: CUDA tensor [B][n][d] fp16/fp32, contiguous.  Returns (and fills) the cache."""
    import torch
    assert blocks.is_cuda and blocks.is_contiguous() and blocks.dim() == 3
    B, n, d = blocks.shape
    if out is None:
        out = Cache.allocate(B, n, d, bits, device=blocks.device)
    if workspace is None:
        workspace = torch.empty(max(eosq_workspace_bytes(B, n, d), 256), dtype=torch.uint8, device=blocks.device)
    st = out.struct()
    rc = lib().eosq_encode(ctx._h, blocks.data_ptr() if B else None, _dtype_code(blocks), B, n, d, bits,
                           ctypes.c_uint64(seed), ctypes.addressof(st), workspace.data_ptr(), workspace.numel(),
                           _stream_ptr(stream))
    _check(rc, "eosq_encode", ctx)
    return out


def eosq_encode_static_max_blocks() -> int:
    return int(lib().eosq_encode_static_max_blocks())


def eosq_encode_static(ctx: Context, blocks, bits: int, seed: int, out: Cache, stream=None) -> Cache:
    """``eosq_encode`` for callers that may not allocate device memory: no workspace argument, the
    library's fixed device array serves as scratch.  ``out`` must be allocated by the caller
    beforehand; at most ``eosq_encode_static_max_blocks()`` blocks per call.  This wrapper itself
    creates no tensor."""
    assert blocks.is_cuda and blocks.is_contiguous() and blocks.dim() == 3
    B, n, d = blocks.shape
    st = out.struct()
    rc = lib().eosq_encode_static(ctx._h, blocks.data_ptr() if B else None, _dtype_code(blocks), B, n, d, bits,
                                  ctypes.c_uint64(seed), ctypes.addressof(st), _stream_ptr(stream))
    if rc == EOSQ_ERR_BUFFER_TOO_SMALL:
        raise EosqError(rc, "eosq_encode_static", lib().eosq_last_cuda_error(ctx._h).decode())
    _check(rc, "eosq_encode_static", ctx)
    return out


def eosq_decode(ctx: Context, cache: Cache, seed: int, out_dtype=None, out=None, stream=None):
    import torch
    out_dtype = out_dtype or torch.float32
    if out is None:
        out = torch.empty((cache.num_blocks, cache.n, cache.d), dtype=out_dtype, device=cache.codes.device)
    st = cache.struct()
    rc = lib().eosq_decode(ctx._h, ctypes.addressof(st), cache.num_blocks, cache.n, cache.d, cache.bits,
                           ctypes.c_uint64(seed), out.data_ptr() if cache.num_blocks else None, _dtype_code(out),
                           _stream_ptr(stream))
    _check(rc, "eosq_decode", ctx)
    return out


def eosq_scores(ctx: Context, kcache: Cache, q, num_kv_heads: int, blocks_per_head: int, head_stride_blocks: int,
                seed: int, scale: Optional[float] = None, out=None, stream=None):
    """q: CUDA fp16 [num_kv_heads][G][d].  Returns fp32 [num_kv_heads][G][blocks_per_head*n]."""
    import torch
    assert q.is_cuda and q.dtype == torch.float16 and q.is_contiguous()
    G = q.shape[1]
    if scale is None:
        scale = 1.0 / float(np.sqrt(kcache.d))
    if out is None:
        out = torch.empty((num_kv_heads, G, blocks_per_head * kcache.n), dtype=torch.float32, device=q.device)
    st = kcache.struct()
    rc = lib().eosq_scores(ctx._h, ctypes.addressof(st), num_kv_heads, blocks_per_head, head_stride_blocks, kcache.n,
                           kcache.d, kcache.bits, ctypes.c_uint64(seed), q.data_ptr(), G, ctypes.c_float(scale),
                           out.data_ptr(), _stream_ptr(stream))
    _check(rc, "eosq_scores", ctx)
    return out


def eosq_encode_host(ctx: Context, host_blocks, bits: int, seed: int, host_out: Cache, arena, stream=None) -> Cache:
    """host_blocks: CPU tensor [B][n][d] (pinned preferred); host_out: Cache of CPU tensors;
    arena: CUDA uint8 tensor of at least eosq_encode_host_arena_bytes()."""
    assert not host_blocks.is_cuda and host_blocks.is_contiguous()
    B, n, d = host_blocks.shape
    st = host_out.struct()
    rc = lib().eosq_encode_host(ctx._h, host_blocks.data_ptr(), _dtype_code(host_blocks), B, n, d, bits,
                                ctypes.c_uint64(seed), ctypes.addressof(st), arena.data_ptr(), arena.numel(),
                                _stream_ptr(stream))
    _check(rc, "eosq_encode_host", ctx)
    return host_out


def eosq_check_status(ctx: Context, cache: Cache, stream=None) -> int:
    """Number of blocks whose status word is non-zero (synchronises the stream)."""
    flagged = ctypes.c_int64(0)
    rc = lib().eosq_check_status(ctx._h, cache.status.data_ptr() if cache.num_blocks else None, cache.num_blocks,
                                 ctypes.byref(flagged), _stream_ptr(stream))
    if rc not in (EOSQ_OK, EOSQ_WARN_BLOCK_STATUS):
        _check(rc, "eosq_check_status", ctx)
    return int(flagged.value)
