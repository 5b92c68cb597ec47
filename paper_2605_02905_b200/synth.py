"""Seeded synthetic KV-cache blocks (spiked model with coloured noise).

Input recipe only: this module draws test and benchmark inputs and holds none of the
compression method's arithmetic.  It serves both the CUDA library's callers and the CPU
oracle's tests, which is why it lives apart from both.

Model (the paper's Eq. "spiked" / "separable" in the appendix, with B diagonal, A = I):

    S_tilde = sum_i theta_i u_i v_i^T + X diag(sigma_j),   X_tj iid N(0, 1/n)

u_i, v_i orthonormal (QR of Gaussians).  theta_i is given as a multiple of the BBP
threshold alpha = 1/sqrt(T(lambda_+)) of the *population* noise model, computed here from the
Silverstein equation of X diag(sigma_j).  Key blocks can carry a few fixed "outlier
channels": columns with a smooth oscillation ten times the noise scale (vertical stripes).
Everything is multiplied by ``value_scale`` at the end so fp16 sees O(0.1 .. 10) values.

Shapes follow the caches the paper measures on (Llama-3.1-8B: 32 layers x 8 KV heads,
Ministral-8B: 36 x 8, head dim 128, fp16); the real caches, which need model weights and a
LongBench passage, are not available offline and these blocks stand in for them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np
import torch


# --------------------------------------------------------------------------- #
# Population noise model: bulk edge and BBP threshold
# --------------------------------------------------------------------------- #

def noise_edge_and_threshold(sigma2: np.ndarray, n: int):
    """Right bulk edge lambda_+ of Z Z^T and the critical spike strength alpha for
    Z = X diag(sigma_j), X (n x d) iid N(0, 1/n).

    The companion Stieltjes transform m (of the n x n matrix Z Z^T) solves
        z(m) = -1/m + (1/n) sum_j sigma_j^2 / (1 + sigma_j^2 m);
    lambda_+ is the minimum of z(m) over m in (-1/max sigma_j^2, 0); the d x d side has
    m_d = (m + (1 - d/n)/z) / (d/n), and alpha = 1/sqrt(lambda_+ m m_d).
    """
    s2 = np.asarray(sigma2, dtype=np.float64)
    d = s2.size
    lo = -1.0 / s2.max() * (1.0 - 1e-12)
    hi = -1e-12

    def dz(m):
        return 1.0 / (m * m) - np.sum((s2 / (1.0 + s2 * m)) ** 2) / n

    for _ in range(200):
        mid = 0.5 * (lo + hi)
        if dz(mid) < 0.0:
            lo = mid
        else:
            hi = mid
    m = 0.5 * (lo + hi)
    lam = -1.0 / m + np.sum(s2 / (1.0 + s2 * m)) / n
    c = d / n
    m_d = (m + (1.0 - c) / lam) / c
    alpha = 1.0 / math.sqrt(lam * m * m_d)
    return float(lam), float(alpha)


# --------------------------------------------------------------------------- #
# Block generator
# --------------------------------------------------------------------------- #

@dataclass
class Workload:
    """A named batch of blocks: blocks[B][n][d] plus what was planted (information only)."""
    name: str
    blocks: torch.Tensor
    n: int
    d: int
    planted_rank: np.ndarray
    is_key: np.ndarray
    meta: dict = field(default_factory=dict)


def _orthonormal(gen, batch, rows, cols, device):
    """Orthonormal columns from a Gaussian draw, by Cholesky-QR in double (two batched calls
    instead of one factorisation per matrix): Q = G L^-T with G^T G = L L^T."""
    g = torch.randn(batch, rows, cols, generator=gen, device=device, dtype=torch.float32).double()
    chol = torch.linalg.cholesky(g.transpose(1, 2) @ g)
    q = torch.linalg.solve_triangular(chol, g.transpose(1, 2), upper=False).transpose(1, 2)
    return q.float()


def spiked_blocks(num_blocks, n, d, *, ranks, theta_mult, sigma_col, alpha, outlier=None,
                  value_scale=None, dtype=torch.float16, device="cpu", seed=0, chunk=512):
    """Draw ``num_blocks`` blocks.

    ranks[B] ints; theta_mult[B][rmax] multiples of alpha (entries past ranks[b] ignored);
    sigma_col[B][d] column noise scales; alpha[B] thresholds; outlier: None or a dict with
    'mask'[B] bool, 'channels'[B][c] int64, 'omega'[B][c], 'phase'[B][c], 'amp'[B].
    """
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    ranks_t = torch.as_tensor(np.asarray(ranks), device=device)
    rmax = max(int(np.max(ranks)) if len(ranks) else 0, 1)
    theta = torch.as_tensor(np.asarray(theta_mult, dtype=np.float32)[:, :rmax], device=device)
    theta = theta * torch.as_tensor(np.asarray(alpha, dtype=np.float32), device=device)[:, None]
    live = torch.arange(rmax, device=device)[None, :] < ranks_t[:, None]
    theta = torch.where(live, theta, torch.zeros_like(theta))
    sig = torch.as_tensor(np.asarray(sigma_col, dtype=np.float32), device=device)
    if value_scale is None:
        value_scale = 0.5 * math.sqrt(n)
    out = torch.empty(num_blocks, n, d, dtype=dtype, device=device)
    tpos = torch.arange(n, device=device, dtype=torch.float32)
    for lo in range(0, num_blocks, chunk):
        hi = min(lo + chunk, num_blocks)
        b = hi - lo
        u = _orthonormal(gen, b, n, rmax, device)
        v = _orthonormal(gen, b, d, rmax, device)
        x = torch.randn(b, n, d, generator=gen, device=device, dtype=torch.float32) / math.sqrt(n)
        blk = x * sig[lo:hi, None, :] + torch.einsum("bnr,br,bdr->bnd", u, theta[lo:hi], v)
        if outlier is not None:
            ch = torch.as_tensor(outlier["channels"][lo:hi], device=device)
            om = torch.as_tensor(np.asarray(outlier["omega"][lo:hi], dtype=np.float32), device=device)
            ph = torch.as_tensor(np.asarray(outlier["phase"][lo:hi], dtype=np.float32), device=device)
            amp = torch.as_tensor(np.asarray(outlier["amp"][lo:hi], dtype=np.float32), device=device)
            msk = torch.as_tensor(np.asarray(outlier["mask"][lo:hi]), device=device)
            stripe = torch.cos(tpos[None, :, None] * om[:, None, :] + ph[:, None, :])  # [b][n][c]
            stripe = stripe * (amp * msk.float())[:, None, None] / math.sqrt(n)
            blk.scatter_add_(2, ch[:, None, :].expand(b, n, ch.shape[1]), stripe)
        out[lo:hi] = (blk * value_scale).to(dtype)
    return out


def pr1_block(seed: int = 0, device="cpu"):
    """The small reference case: one 256 x 128 fp32 block, white noise N(0, 1/256), four
    spikes at {8, 4, 2, 0.5} x the BBP threshold (the last one is below it and must be
    rejected)."""
    n, d = 256, 128
    lam, alpha = noise_edge_and_threshold(np.ones(d), n)
    blocks = spiked_blocks(1, n, d, ranks=[4], theta_mult=[[8.0, 4.0, 2.0, 0.5]],
                           sigma_col=np.ones((1, d)), alpha=[alpha], value_scale=1.0,
                           dtype=torch.float32, device=device, seed=seed)
    return Workload("pr1", blocks, n, d, np.array([4]), np.array([False]),
                    dict(alpha=alpha, lambda_plus=lam, theta=[8 * alpha, 4 * alpha, 2 * alpha, 0.5 * alpha]))


def kv_cache_blocks(name, *, layers, kv_heads, tokens, n, d=128, rank_lo=2, rank_hi=16,
                    theta_lo=1.5, theta_hi=20.0, noise_frac=0.0, key_outliers=4,
                    fixed_theta=None, device="cpu", seed=0, max_blocks=None, dtype=torch.float16):
    """Blocks of a [layers][kv_heads][K|V][tokens][d] cache, in that order, cut every n tokens.

    Per (layer, head, K|V) one column-scale vector sigma_j (log-uniform in [0.5, 2]) is fixed
    across its blocks; per block the planted rank is uniform in {rank_lo..rank_hi} and
    theta_i log-uniform in [theta_lo, theta_hi] x alpha; a fraction ``noise_frac`` of blocks
    is pure noise; key blocks add ``key_outliers`` fixed channels per head with an
    oscillation of ten times the median noise scale.  ``fixed_theta`` (a list of multiples
    of alpha) overrides the random ranks and strengths.  ``max_blocks`` keeps a prefix.
    """
    rng = np.random.default_rng(seed)
    per_stream = tokens // n
    streams = layers * kv_heads * 2
    total = streams * per_stream
    if max_blocks is not None:
        total = min(total, int(max_blocks))
    n_streams_used = (total + per_stream - 1) // per_stream
    sig_stream = np.exp(rng.uniform(math.log(0.5), math.log(2.0), size=(n_streams_used, d)))
    alpha_stream = np.array([noise_edge_and_threshold(s * s, n)[1] for s in sig_stream])
    stream_of = np.arange(total) // per_stream
    is_key = (stream_of % 2) == 0
    rcap = rank_hi if fixed_theta is None else len(fixed_theta)
    if fixed_theta is None:
        ranks = rng.integers(rank_lo, rank_hi + 1, size=total)
        mult = np.exp(rng.uniform(math.log(theta_lo), math.log(theta_hi), size=(total, max(rcap, 1))))
        mult = -np.sort(-mult, axis=1)
    else:
        ranks = np.full(total, len(fixed_theta))
        mult = np.tile(np.asarray(fixed_theta, dtype=np.float64)[None, :], (total, 1))
    if noise_frac > 0:
        ranks = np.where(rng.uniform(size=total) < noise_frac, 0, ranks)
    outlier = None
    if key_outliers > 0:
        ch_stream = np.stack([rng.choice(d, size=key_outliers, replace=False) for _ in range(n_streams_used)])
        om_stream = rng.uniform(0.002, 0.02, size=(n_streams_used, key_outliers))
        ph_stream = rng.uniform(0, 2 * math.pi, size=(n_streams_used, key_outliers))
        start = (np.arange(total) % per_stream) * n  # token offset of the block in its stream
        outlier = dict(
            mask=is_key,
            channels=ch_stream[stream_of].astype(np.int64),
            omega=om_stream[stream_of],
            phase=ph_stream[stream_of] + om_stream[stream_of] * start[:, None],
            amp=10.0 * np.median(sig_stream, axis=1)[stream_of],
        )
    blocks = spiked_blocks(total, n, d, ranks=ranks, theta_mult=mult, sigma_col=sig_stream[stream_of],
                           alpha=alpha_stream[stream_of], outlier=outlier, dtype=dtype, device=device,
                           seed=seed + 1)
    return Workload(name, blocks, n, d, ranks, is_key,
                    dict(layers=layers, kv_heads=kv_heads, tokens=tokens, blocks_per_stream=per_stream))


# The benchmark configurations, by name.
def llama_1layer(device="cpu", seed=1, max_blocks=None):
    """One Llama-3.1-8B-shaped layer: 8 KV heads x {K,V}, T = 8192, n = 1024 (128 blocks)."""
    return kv_cache_blocks("llama31_8b_1layer_T8192", layers=1, kv_heads=8, tokens=8192, n=1024,
                           device=device, seed=seed, max_blocks=max_blocks)


def llama_32k(device="cpu", seed=2, max_blocks=None):
    """Full Llama-3.1-8B-shaped cache: 32 x 8 x {K,V}, T = 32768, n = 1024 (16384 blocks, 4 GiB)."""
    return kv_cache_blocks("llama31_8b_T32768", layers=32, kv_heads=8, tokens=32768, n=1024,
                           device=device, seed=seed, max_blocks=max_blocks)


def ministral_64k(device="cpu", seed=3, max_blocks=None):
    """Ministral-8B-shaped cache: 36 x 8 x {K,V}, T = 65536, rank up to 32, 5% pure-noise blocks."""
    return kv_cache_blocks("ministral_8b_T65536", layers=36, kv_heads=8, tokens=65536, n=1024,
                           rank_lo=1, rank_hi=32, noise_frac=0.05, device=device, seed=seed,
                           max_blocks=max_blocks)


def sweep_point(n, device="cpu", seed=4, max_blocks=None):
    """Sweep shape: 1 layer x 8 KV heads, T = 131072, four spikes at {0.9, 1.05, 1.5, 5} x alpha."""
    return kv_cache_blocks(f"sweep_n{n}", layers=1, kv_heads=8, tokens=131072, n=n,
                           fixed_theta=[5.0, 1.5, 1.05, 0.9], device=device, seed=seed,
                           max_blocks=max_blocks)


def queries(num_kv_heads, G, d=128, device="cpu", seed=7):
    """Query vectors [num_kv_heads][G][d], iid N(0,1), fp16 (G = query heads per KV head x batch)."""
    gen = torch.Generator(device=device)
    gen.manual_seed(int(seed))
    return torch.randn(num_kv_heads, G, d, generator=gen, device=device, dtype=torch.float32).to(torch.float16)
