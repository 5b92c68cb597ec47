"""CPU oracle for the eOptShrinkQ hot path -- TEST INFRASTRUCTURE, NOT THE PRODUCT.

Thin numpy/ctypes front end over ``eosq_oracle.c`` (double precision, plain loops).
Only tests, the smoke check and the benchmark's CPU-baseline leg may import this
package; the CUDA library never does, and shares no code with it.

Every function names the passage of the paper it follows in the C source.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from pathlib import Path

import numpy as np

_HERE = Path(__file__).resolve().parent
_SRC = _HERE / "eosq_oracle.c"
_LIB = _HERE / "liboracle.so"

_dp = ctypes.POINTER(ctypes.c_double)
_u8p = ctypes.POINTER(ctypes.c_uint8)
_i32p = ctypes.POINTER(ctypes.c_int32)


def build(force: bool = False) -> Path:
    """Compile the C oracle into ``liboracle.so`` next to its source (gcc, OpenMP over blocks)."""
    if force or not _LIB.exists() or _LIB.stat().st_mtime < _SRC.stat().st_mtime:
        tmp = _LIB.with_suffix(f".tmp{os.getpid()}.so")
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fPIC", "-shared", "-fopenmp", "-o", str(tmp), str(_SRC), "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(str(_LIB))
        _lib.orc_codebook_distortion.restype = ctypes.c_double
    return _lib


def _d(a):
    return a.ctypes.data_as(_dp)


def _f64(a):
    return np.ascontiguousarray(a, dtype=np.float64)


def num_threads() -> int:
    return int(_load().orc_num_threads())


def pilot_k(d: int) -> int:
    return int(_load().orc_pilot_k(int(d)))


def codebook(bits: int, d: int):
    """Lloyd-Max centroids (2^bits, ascending) and midpoint thresholds for N(0, 1/d)."""
    c = np.zeros(1 << bits)
    t = np.zeros((1 << bits) - 1)
    _load().orc_codebook(int(bits), int(d), _d(c), _d(t))
    return c, t


def codebook_distortion(bits: int, d: int, centroids) -> float:
    c = _f64(centroids)
    return float(_load().orc_codebook_distortion(int(bits), int(d), _d(c)))


def gaussian_matrix(d: int, seed: int):
    a = np.zeros((d, d))
    _load().orc_gaussian_matrix(int(d), ctypes.c_uint64(seed), _d(a))
    return a


def rotation(d: int, seed: int):
    """Seeded Haar rotation Pi (d x d, row-major, z = Pi u)."""
    pi = np.zeros((d, d))
    _load().orc_rotation(int(d), ctypes.c_uint64(seed), _d(pi))
    return pi


def svd(S):
    """One-sided Jacobi SVD of an n x d block (n >= d): sigma (desc), U (n x d), V (d x d)."""
    S = _f64(S)
    n, d = S.shape
    assert n >= d
    sigma = np.zeros(d)
    U = np.zeros((n, d))
    V = np.zeros((d, d))
    sweeps = _load().orc_svd(n, d, _d(S), _d(sigma), _d(U), _d(V))
    return sigma, U, V, int(sweeps)


def eoptshrink_spectrum(n: int, d: int, sigma, k: int = 0):
    """Algorithm 2 on a spectrum: bulk edge, rank, imputed atoms, D-transform, shrunk values."""
    sigma = _f64(sigma)
    q = min(n, d)
    assert sigma.shape == (q,)
    scal = np.zeros(5)
    arrs = {name: np.zeros(q) for name in ("atoms", "m1", "m2", "T", "Tp", "dhat", "a1", "a2", "phi")}
    r = _load().orc_eoptshrink_spectrum(
        int(n), int(d), _d(sigma), int(k), _d(scal),
        _d(arrs["atoms"]), _d(arrs["m1"]), _d(arrs["m2"]), _d(arrs["T"]), _d(arrs["Tp"]),
        _d(arrs["dhat"]), _d(arrs["a1"]), _d(arrs["a2"]), _d(arrs["phi"]),
    )
    out = dict(arrs)
    out.update(status=int(r), k=int(scal[0]), lambda_plus=float(scal[1]), rank=int(scal[2]),
               margin=float(scal[3]), clamped=int(scal[4]))
    return out


def residual(S, Vr, coef):
    """R = S - sum_i coef_i (S v_i) v_i^T, Vr is d x r (columns v_i).  Also the stored left factor."""
    S = _f64(S)
    n, d = S.shape
    Vr = _f64(Vr).reshape(d, -1)
    r = Vr.shape[1]
    coef = _f64(coef).reshape(r)
    R = np.zeros((n, d))
    P = np.zeros((max(r, 1), n))
    _load().orc_residual(n, d, r, _d(S), _d(Vr), _d(coef), _d(R), _d(P))
    return R, P[:r]


def tq_rows(R, Pi, thresholds, bits: int):
    """Norm separation, rotation and Lloyd-Max codes of every row (Algorithm 1)."""
    R = _f64(R)
    n, d = R.shape
    Pi = _f64(Pi)
    thr = _f64(thresholds)
    rho = np.zeros(n)
    z = np.zeros((n, d))
    codes = np.zeros((n, d), dtype=np.uint8)
    _load().orc_tq_rows(n, d, int(bits), _d(R), _d(Pi), _d(thr), _d(rho), _d(z),
                        codes.ctypes.data_as(_u8p))
    return rho, z, codes


def pack(codes, bits: int):
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    n, d = codes.shape
    out = np.zeros((n, (d * bits + 7) // 8), dtype=np.uint8)
    _load().orc_pack(n, d, int(bits), codes.ctypes.data_as(_u8p), out.ctypes.data_as(_u8p))
    return out


def unpack(packed, d: int, bits: int):
    packed = np.ascontiguousarray(packed, dtype=np.uint8)
    n = packed.shape[0]
    out = np.zeros((n, d), dtype=np.uint8)
    _load().orc_unpack(n, int(d), int(bits), packed.ctypes.data_as(_u8p), out.ctypes.data_as(_u8p))
    return out


def decode(codes, rho, Pfac, Vfac, Pi, centroids):
    """x_hat = Pfac^T Vfac + rho * (centroids[codes] Pi); Pfac [r][n], Vfac [r][d] as stored."""
    codes = np.ascontiguousarray(codes, dtype=np.uint8)
    n, d = codes.shape
    Pfac = _f64(Pfac).reshape(-1, n)
    r = Pfac.shape[0]
    Vfac = _f64(Vfac).reshape(r, d)
    if r == 0:
        Pfac = np.zeros((1, n))
        Vfac = np.zeros((1, d))
    rho = _f64(rho)
    Pi = _f64(Pi)
    cen = _f64(centroids)
    X = np.zeros((n, d))
    _load().orc_decode(n, d, 0, r, codes.ctypes.data_as(_u8p), _d(rho), _d(Pfac), _d(Vfac),
                       _d(Pi), _d(cen), _d(X))
    return X


def scores(X, Y, scale: float):
    """scores[g][t] = scale * <y_g, x_t>."""
    X = _f64(X)
    Y = _f64(Y)
    n, d = X.shape
    G = Y.shape[0]
    out = np.zeros((G, n))
    _load().orc_scores(n, d, G, _d(X), _d(Y), ctypes.c_double(scale), _d(out))
    return out


def encode_blocks(S, bits: int, seed: int, rmax: int = 16):
    """Algorithm 3 on every block of S [B][n][d] (any float dtype; widened exactly to double).

    Returns a dict of per-block arrays: sigma [B][d], k, lambda_plus, rank, margin, clamped,
    phi/dhat/a1/a2 [B][d], V [B][rmax][d], P [B][rmax][n], rho [B][n], z [B][n][d],
    codes [B][n][d], packed [B][n][d*bits/8], plus the rotation and codebook used.
    """
    S = _f64(S)
    if S.ndim == 2:
        S = S[None]
    B, n, d = S.shape
    Pi = rotation(d, seed)
    cen, thr = codebook(bits, d)
    row_bytes = (d * bits + 7) // 8
    out = dict(
        sigma=np.zeros((B, d)), scal=np.zeros((B, 5)), phi=np.zeros((B, d)), dhat=np.zeros((B, d)),
        a1=np.zeros((B, d)), a2=np.zeros((B, d)), V=np.zeros((B, rmax, d)), P=np.zeros((B, rmax, n)),
        rho=np.zeros((B, n)), z=np.zeros((B, n, d)), codes=np.zeros((B, n, d), dtype=np.uint8),
        packed=np.zeros((B, n, row_bytes), dtype=np.uint8), ranks=np.zeros(B, dtype=np.int32),
    )
    bad = _load().orc_encode_batch(
        ctypes.c_int64(B), n, d, int(bits), int(rmax), _d(S), _d(Pi), _d(thr),
        _d(out["sigma"]), _d(out["scal"]), _d(out["phi"]), _d(out["dhat"]), _d(out["a1"]), _d(out["a2"]),
        _d(out["V"]), _d(out["P"]), _d(out["rho"]), _d(out["z"]),
        out["codes"].ctypes.data_as(_u8p), out["packed"].ctypes.data_as(_u8p),
        out["ranks"].ctypes.data_as(_i32p),
    )
    if bad:
        raise RuntimeError(f"oracle: {bad} block(s) outside the supported range (3k+1 > min(n,d) or rank > rmax)")
    scal = out.pop("scal")
    out.update(k=scal[:, 0].astype(np.int32), lambda_plus=scal[:, 1].copy(), rank=out.pop("ranks"),
               margin=scal[:, 3].copy(), clamped=scal[:, 4].astype(np.int32),
               Pi=Pi, centroids=cen, thresholds=thr, bits=bits, n=n, d=d)
    return out


def stored(enc, b: int):
    """What Algorithm 3's Store line keeps for block b, rounded as the format states:
    fp16 norms, fp16 left/right factors (rows [0, rank)), packed codes."""
    r = int(enc["rank"][b])
    return dict(
        rank=r,
        norms=enc["rho"][b].astype(np.float16),
        P=enc["P"][b, :r].astype(np.float16),
        V=enc["V"][b, :r].astype(np.float16),
        packed=enc["packed"][b],
    )


def decode_stored(enc, b: int):
    """Reconstruction of block b from its stored (rounded) values."""
    st = stored(enc, b)
    codes = unpack(st["packed"], enc["d"], enc["bits"])
    return decode(codes, st["norms"].astype(np.float64), st["P"].astype(np.float64),
                  st["V"].astype(np.float64), enc["Pi"], enc["centroids"])


def bits_per_entry(b: int, rank: float, n: int, d: int, b_s: float, prod: bool = False,
                   count_norms: bool = False, count_sigma: bool = False) -> float:
    """Algorithm 3's bit budget: b + rank (n + d) b_s / (n d) (+1 with the QJL bit); Remark 3.1's
    two small shared costs (16/d for the fp16 row norm, 16 rank / (n d) for the shrunk values)
    are added on request."""
    bits = b + rank * (n + d) * b_s / (n * d) + (1.0 if prod else 0.0)
    if count_norms:
        bits += 16.0 / d
    if count_sigma:
        bits += 16.0 * rank / (n * d)
    return bits
