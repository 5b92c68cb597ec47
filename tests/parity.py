"""Shared comparison logic of the GPU parity tests: CUDA library vs CPU oracle on the same
seeded blocks.  Tolerances are the ones the task states:

  * ranks and packed codes bit-exact, except codes whose rotated coordinate lies within
    1e-5 (relative to the coordinate scale 1/sqrt(d)) of a decision threshold -- counted;
  * singular values and shrunk values within 1e-4 relative;
  * reconstruction within 1e-4 relative Frobenius error; scores within 1e-3 relative.

Stages amplify each other (a 1e-7 change of a right vector moves every residual coordinate),
so codes are compared twice: against the oracle's quantiser fed the library's own factors
(strict), and against the oracle end to end (counted, with a bound).
"""
from __future__ import annotations

import math

import numpy as np
import torch

import oracle
import paper_2605_02905_b200 as eosq

BAND = 1e-5          # relative half-width of the exemption band around a threshold
SIGMA_TOL = 1e-4     # singular values, shrunk values, bulk edge
DECODE_TOL = 1e-4    # relative Frobenius, decode of identical stored bytes
SCORE_TOL = 1e-3
RANK_MARGIN = 1e-4   # blocks whose rank test is this close to its cut are compared separately


def to_numpy_cache(cache: eosq.Cache) -> dict:
    out = {}
    for name in ("codes", "norms", "rank", "sigma", "phi", "P", "V", "status", "eig", "lambda_plus", "vr32", "coef"):
        t = getattr(cache, name)
        out[name] = None if t is None else t.detach().cpu().numpy()
    return out


def compare_encode(blocks_cpu: torch.Tensor, cache: eosq.Cache, bits: int, seed: int, blocks_idx=None, enc=None):
    """Compare the library's cache with the oracle on the given blocks.  Returns a report dict and
    raises AssertionError on any violation."""
    g = to_numpy_cache(cache)
    B, n, d = blocks_cpu.shape
    idx = list(range(B)) if blocks_idx is None else list(blocks_idx)
    S_all = blocks_cpu.double().numpy()
    if enc is None:
        enc = oracle.encode_blocks(S_all[idx], bits, seed)
    cen, thr, Pi = enc["centroids"], enc["thresholds"], enc["Pi"]
    band = BAND / math.sqrt(d)
    rep = dict(blocks=len(idx), near_threshold_blocks=0, rank_mismatch=0, codes=0, staged_mismatch_in_band=0,
               staged_mismatch_out_band=0, e2e_mismatch_in_band=0, e2e_mismatch_out_band=0,
               max_sigma_rel=0.0, max_phi_rel=0.0, max_lowrank_rel=0.0, flagged=0)
    for k, b in enumerate(idx):
        S = S_all[b]
        o_rank = int(enc["rank"][k])
        g_rank = int(g["rank"][b])
        near = enc["margin"][k] < RANK_MARGIN
        rep["near_threshold_blocks"] += int(near)
        rep["flagged"] += int(g["status"][b] != 0)
        # --- gate 1: spectrum, edge, rank, shrinkage
        sig_o = enc["sigma"][k]
        live = sig_o > 1e-6 * sig_o[0] if sig_o[0] > 0 else np.zeros(d, bool)
        if live.any() and g["eig"] is not None:   # the whole spectrum, when the cache asked for it
            sig_g = np.sqrt(np.maximum(g["eig"][b].astype(np.float64), 0.0))
            rel = np.abs(sig_g[live] - sig_o[live]) / sig_o[live]
            rep["max_sigma_rel"] = max(rep["max_sigma_rel"], float(rel.max()))
            assert rel.max() < SIGMA_TOL, f"block {b}: singular values off by {rel.max():.3e}"
        if live.any():
            assert abs(g["lambda_plus"][b] / enc["lambda_plus"][k] - 1) < SIGMA_TOL
        if g_rank != o_rank:
            rep["rank_mismatch"] += 1
            assert near, f"block {b}: rank {g_rank} vs oracle {o_rank} (margin {enc['margin'][k]:.3e})"
            continue
        r = o_rank
        if r:
            rel_s = np.abs(g["sigma"][b, :r] / sig_o[:r] - 1).max()
            rel_p = np.abs(g["phi"][b, :r] / enc["phi"][k, :r] - 1).max()
            rep["max_sigma_rel"] = max(rep["max_sigma_rel"], float(rel_s))
            rep["max_phi_rel"] = max(rep["max_phi_rel"], float(rel_p))
            assert rel_s < SIGMA_TOL and rel_p < SIGMA_TOL, f"block {b}: sigma {rel_s:.2e} phi {rel_p:.2e}"
        assert np.all(g["sigma"][b, r:] == 0) and np.all(g["phi"][b, r:] == 0)
        assert np.all(g["V"][b, r:] == 0)
        # --- low-rank part as stored (signs of singular vectors are free: compare the product)
        if r:
            low_g = g["P"][b, :r].astype(np.float64).T @ g["V"][b, :r].astype(np.float64)
            low_o = enc["P"][k, :r].T @ enc["V"][k, :r]
            rel_l = np.linalg.norm(low_g - low_o) / np.linalg.norm(low_o)
            rep["max_lowrank_rel"] = max(rep["max_lowrank_rel"], float(rel_l))
            assert rel_l < 2e-3, f"block {b}: stored low-rank part off by {rel_l:.2e}"  # fp16 storage rounding
        # --- gate 2: the oracle's quantiser fed the library's own (unrounded) factors
        g_codes = oracle.unpack(g["codes"][b], d, bits)
        Rg, _ = oracle.residual(S, g["vr32"][b, :r].astype(np.float64).T, g["coef"][b, :r].astype(np.float64))
        rho_s, z_s, codes_s = oracle.tq_rows(Rg, Pi, thr, bits)
        dist_s = np.abs(z_s[:, :, None] - thr[None, None, :]).min(axis=2)
        mism = g_codes != codes_s
        rep["codes"] += mism.size
        rep["staged_mismatch_in_band"] += int((mism & (dist_s <= band)).sum())
        out_band = int((mism & (dist_s > band)).sum())
        rep["staged_mismatch_out_band"] += out_band
        assert out_band == 0, f"block {b}: {out_band} codes differ outside the 1e-5 band (staged)"
        # norms: fp16 rounding of a value known to ~1e-6 relative may land on the neighbouring fp16
        norms_g = g["norms"][b].astype(np.float64)
        assert np.all(np.abs(norms_g - rho_s) <= np.maximum(rho_s, 6.2e-5) * 2.0 ** -10), f"block {b}: norms"
        # --- gate 3: end to end against the oracle's own factors (counted)
        dist_o = np.abs(enc["z"][k][:, :, None] - thr[None, None, :]).min(axis=2)
        mism_o = g_codes != enc["codes"][k]
        rep["e2e_mismatch_in_band"] += int((mism_o & (dist_o <= band)).sum())
        rep["e2e_mismatch_out_band"] += int((mism_o & (dist_o > band)).sum())
    rep["e2e_out_band_fraction"] = rep["e2e_mismatch_out_band"] / max(rep["codes"], 1)
    return rep, enc


def oracle_decode_of_stored(g: dict, b: int, n: int, d: int, bits: int, Pi, cen):
    """The oracle's reconstruction of block b from the bytes the library stored."""
    r = int(g["rank"][b])
    codes = oracle.unpack(g["codes"][b], d, bits)
    return oracle.decode(codes, g["norms"][b].astype(np.float64), g["P"][b, :r].astype(np.float64),
                         g["V"][b, :r].astype(np.float64), Pi, cen)


def compare_decode(cache: eosq.Cache, decoded: torch.Tensor, bits: int, seed: int, blocks_idx=None, tol=DECODE_TOL):
    g = to_numpy_cache(cache)
    B, n, d = decoded.shape
    Pi = oracle.rotation(d, seed)
    cen, _ = oracle.codebook(bits, d)
    worst = 0.0
    for b in (range(B) if blocks_idx is None else blocks_idx):
        X = oracle_decode_of_stored(g, b, n, d, bits, Pi, cen)
        Xg = decoded[b].double().cpu().numpy()
        den = np.linalg.norm(X)
        rel = np.linalg.norm(Xg - X) / den if den > 0 else np.abs(Xg).max()
        worst = max(worst, float(rel))
        assert rel < tol, f"block {b}: decode off by {rel:.3e}"
    return worst


def compare_scores(cache: eosq.Cache, q: torch.Tensor, scores: torch.Tensor, heads, bph, head_stride, bits, seed,
                   scale, pairs=None):
    """scores [heads][G][bph*n] against scale * <q, oracle decode of the stored bytes>."""
    g = to_numpy_cache(cache)
    n, d = cache.n, cache.d
    Pi = oracle.rotation(d, seed)
    cen, _ = oracle.codebook(bits, d)
    qn = q.double().cpu().numpy()
    sg = scores.double().cpu().numpy()
    worst = 0.0
    todo = pairs if pairs is not None else [(h, j) for h in range(heads) for j in range(bph)]
    for h, j in todo:
        b = h * head_stride + j
        X = oracle_decode_of_stored(g, b, n, d, bits, Pi, cen)
        ref = oracle.scores(X, qn[h], scale)                      # [G][n]
        got = sg[h][:, j * n:(j + 1) * n]
        floor = scale * np.linalg.norm(qn[h], axis=1)[:, None] * np.linalg.norm(X, axis=1)[None, :] / math.sqrt(d)
        rel = np.abs(got - ref) / (np.abs(ref) + floor + 1e-30)
        worst = max(worst, float(rel.max()))
        assert rel.max() < SCORE_TOL, f"head {h} block {j}: scores off by {rel.max():.3e}"
    return worst
