"""Pins for the CPU oracle: every check compares it with something other than itself --
values the paper prints, closed forms, library routines on special cases, brute force."""
import math

import numpy as np
import pytest
from scipy import integrate, stats

import oracle
from paper_2605_02905_b200 import synth

EDGE_C = 1.0 / (2.0 ** (2.0 / 3.0) - 1.0)


# --------------------------------------------------------------------------- #
# Codebook (Algorithm 1 REQUIRE; Sec. 2.2 item 3)
# --------------------------------------------------------------------------- #

def test_one_bit_centroids_closed_form():
    for d in (64, 128):
        c, t = oracle.codebook(1, d)
        assert np.allclose(c, np.array([-1.0, 1.0]) * math.sqrt(2.0 / math.pi) / math.sqrt(d), rtol=0, atol=1e-14)
        assert abs(t[0]) < 1e-15


@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_codebook_is_a_lloyd_max_fixed_point(bits):
    """Independent check by numerical quadrature: each centroid is the conditional mean of
    its cell under N(0, 1/d) and each threshold the midpoint of its neighbours."""
    d = 128
    s = 1.0 / math.sqrt(d)
    c, t = oracle.codebook(bits, d)
    assert np.all(np.diff(c) > 0)
    assert np.allclose(c, -c[::-1], atol=1e-14)
    assert np.allclose(t, 0.5 * (c[:-1] + c[1:]), atol=1e-16)
    edges = np.concatenate([[-np.inf], t, [np.inf]])
    for i in range(len(c)):
        num = integrate.quad(lambda x: x * stats.norm.pdf(x, scale=s), edges[i], edges[i + 1], epsabs=1e-15)[0]
        den = integrate.quad(lambda x: stats.norm.pdf(x, scale=s), edges[i], edges[i + 1], epsabs=1e-15)[0]
        assert abs(num / den - c[i]) < 1e-9 * s


@pytest.mark.parametrize("bits,classical", [(1, 0.3634), (2, 0.1175), (3, 0.03454), (4, 0.009497)])
def test_distortion_matches_quadrature_and_classical_table(bits, classical):
    d = 128
    s = 1.0 / math.sqrt(d)
    c, t = oracle.codebook(bits, d)
    D = oracle.codebook_distortion(bits, d, c)
    edges = np.concatenate([[-np.inf], t, [np.inf]])
    quad = sum(
        integrate.quad(lambda x, ci=c[i]: (x - ci) ** 2 * stats.norm.pdf(x, scale=s), edges[i], edges[i + 1], epsabs=1e-16)[0]
        for i in range(len(c))
    ) / (s * s)
    assert abs(D - quad) < 1e-9
    # Max's classical table values (4 significant digits; the 16-level entry is known to 3)
    assert abs(D - classical) < 5e-4 * classical + 5e-6


def test_distortion_matches_paper_tqmse_rows(golden):
    """TQ_MSE's relative L2 error is data independent and equals sqrt(D_b) (Tables 1-4)."""
    for bits in (2, 3, 4):
        c, _ = oracle.codebook(bits, 128)
        pct = 100.0 * math.sqrt(oracle.codebook_distortion(bits, 128, c))
        assert abs(pct - golden[f"tqmse_l2_percent_b{bits}"]) < 0.25


# --------------------------------------------------------------------------- #
# Rotation (Algorithm 1: Haar Pi)
# --------------------------------------------------------------------------- #

@pytest.mark.parametrize("d,seed", [(128, 0), (128, 12345), (64, 7), (16, 3)])
def test_rotation_orthogonal_and_equals_library_qr(d, seed):
    Pi = oracle.rotation(d, seed)
    assert np.abs(Pi.T @ Pi - np.eye(d)).max() < 1e-13
    assert np.abs(Pi @ Pi.T - np.eye(d)).max() < 1e-13
    assert abs(abs(np.linalg.det(Pi)) - 1.0) < 1e-12
    A = oracle.gaussian_matrix(d, seed)
    Q, R = np.linalg.qr(A)
    Q = Q * np.sign(np.diag(R))[None, :]
    assert np.abs(Q - Pi).max() < 1e-12
    # Q^T A must be upper triangular with positive diagonal
    Rr = Pi.T @ A
    assert np.abs(np.tril(Rr, -1)).max() < 1e-12
    assert np.all(np.diag(Rr) > 0)


def test_gaussian_generator_statistics_and_seeding():
    A = oracle.gaussian_matrix(128, 0)
    B = oracle.gaussian_matrix(128, 1)
    assert abs(A.mean()) < 0.03 and abs(A.std() - 1.0) < 0.03
    assert stats.kstest(A.ravel(), "norm").pvalue > 1e-3
    assert np.abs(A - B).max() > 1.0
    assert np.array_equal(A, oracle.gaussian_matrix(128, 0))
    # prefix property of a counter-based generator with row-major counters: none across d
    assert not np.array_equal(oracle.gaussian_matrix(64, 0), A[:64, :64])


def test_rotation_is_haar_like():
    """First column of a Haar matrix is uniform on the sphere: coordinates ~ N(0, 1/d)."""
    cols = np.concatenate([oracle.rotation(64, s)[:, 0] for s in range(40)])
    assert stats.kstest(cols * math.sqrt(64), "norm").pvalue > 1e-3


# --------------------------------------------------------------------------- #
# Constants and bit accounting (Algorithm 2 REQUIRE / Step 1; Remark 3.1; Algorithm 3)
# --------------------------------------------------------------------------- #

def test_pilot_parameter(golden):
    assert oracle.pilot_k(128) == golden["pilot_k_d128"]
    assert oracle.pilot_k(64) == golden["pilot_k_d64"]
    assert abs(EDGE_C - 1.70241) < 1e-5


def test_bits_per_entry(golden):
    assert abs(oracle.bits_per_entry(0, 1, 128, 128, 4) - golden["svd1_overhead_bits_n128_d128_bs4"]) < 0.005
    assert abs(oracle.bits_per_entry(0, 5.6, 128, 128, 4) - golden["eoptshrinkq_overhead_bits_rbar5p6"]) < 0.005
    assert oracle.bits_per_entry(2, 0, 128, 128, 4, count_norms=True) - 2 == golden["norm_bits_per_entry_d128"]
    assert oracle.bits_per_entry(2, 3, 128, 128, 4, prod=True) == oracle.bits_per_entry(2, 3, 128, 128, 4) + 1


# --------------------------------------------------------------------------- #
# SVD against the library routine
# --------------------------------------------------------------------------- #

@pytest.mark.parametrize("n,d,seed", [(256, 128, 0), (128, 128, 1), (40, 16, 2), (300, 64, 3)])
def test_svd_matches_lapack(n, d, seed):
    rng = np.random.default_rng(seed)
    S = rng.standard_normal((n, d)) @ np.diag(np.exp(rng.uniform(-2, 2, d)))
    S[:, 3] += 30 * np.cos(0.01 * np.arange(n))
    sig, U, V, _ = oracle.svd(S)
    ref = np.linalg.svd(S, compute_uv=False)
    assert np.all(np.diff(sig) <= 0)
    assert np.abs(sig - ref).max() < 1e-12 * ref[0]
    assert np.abs(sig / ref - 1).max() < 1e-10
    assert np.abs(U.T @ U - np.eye(d)).max() < 1e-12
    assert np.abs(V.T @ V - np.eye(d)).max() < 1e-12
    assert np.abs((U * sig) @ V.T - S).max() < 1e-11 * ref[0]


# --------------------------------------------------------------------------- #
# Algorithm 2 on a hand-worked spectrum: pins every index of Steps 1-3
# --------------------------------------------------------------------------- #

def _hand_case(n, d):
    """lambda = [100, 9, 8, 7, 6, 5, 4, 3], k forced to 2.  Worked by hand:
    Step 1: lambda_3 = 8, lambda_5 = 6  -> lambda_+ = 8 + 2 E;  cut = 8^(-1/3) = 1/2; only
    lambda_1 passes -> rank 1.  Step 2: lambda_{k+r+1} = lambda_4 = 7, lambda_{2k+r+1} =
    lambda_6 = 5; atoms j=1,2: 7 + (1 - (j/2)^(2/3)) * 2 E, then the observed lambda_4..8."""
    lam = np.array([100.0, 9, 8, 7, 6, 5, 4, 3])
    lam_plus = 8 + 2 * EDGE_C
    atoms = np.array([7 + (1 - 0.5 ** (2.0 / 3.0)) * 2 * EDGE_C, 7.0, 7.0, 6.0, 5.0, 4.0, 3.0])
    z = 100.0
    ms = np.mean(1.0 / (atoms - z))
    msp = np.mean(1.0 / (atoms - z) ** 2)
    q, Q = min(n, d), max(n, d)
    ml = (q / Q) * ms - (1 - q / Q) / z
    mlp = (q / Q) * msp + (1 - q / Q) / z ** 2
    m1, m1p, m2, m2p = (ml, mlp, ms, msp) if n >= d else (ms, msp, ml, mlp)
    T = z * m1 * m2
    Tp = m1 * m2 + z * (m1p * m2 + m1 * m2p)
    dhat = 1 / math.sqrt(T)
    a1 = m1 * T / Tp
    a2 = m2 * T / Tp
    return lam, lam_plus, atoms, m1, m2, T, Tp, dhat, a1, a2, dhat * math.sqrt(a1 * a2)


@pytest.mark.parametrize("n,d", [(8, 8), (16, 8)])
def test_algorithm2_hand_worked_spectrum(n, d):
    lam, lam_plus, atoms, m1, m2, T, Tp, dhat, a1, a2, phi = _hand_case(n, d)
    r = oracle.eoptshrink_spectrum(n, d, np.sqrt(lam), k=2)
    assert r["k"] == 2 and r["rank"] == 1
    assert abs(r["lambda_plus"] - lam_plus) < 1e-13
    assert abs(r["margin"] - min(abs(lam / lam_plus - 1 - 0.5))) < 1e-13
    assert np.allclose(r["atoms"][1:], atoms, rtol=0, atol=1e-13)
    for name, val in (("m1", m1), ("m2", m2), ("T", T), ("Tp", Tp), ("dhat", dhat), ("a1", a1), ("a2", a2), ("phi", phi)):
        assert abs(r[name][0] - val) < 1e-13 * max(1.0, abs(val)), name
    assert m1 < 0 and m2 < 0 and T > 0 and Tp < 0 and 0 < a1 < 1 and 0 < a2 < 1
    assert np.all(r["phi"][1:] == 0)


def test_algorithm2_rejects_too_small_spectrum():
    assert oracle.eoptshrink_spectrum(8, 8, np.sqrt(np.arange(8, 0, -1.0)), k=3)["status"] == -1


# --------------------------------------------------------------------------- #
# White-noise special case: closed forms (Sec. 2.3: MP law, BBP transition; Eq. 6)
# --------------------------------------------------------------------------- #

def _white_closed_form(theta, c):
    lam = (1 + theta ** 2) * (c + theta ** 2) / theta ** 2
    phi = math.sqrt((lam - c - 1) ** 2 - 4 * c) / math.sqrt(lam)
    # noise variance 1/n with n rows: the row-side (left, u) overlap has theta^2 in the
    # denominator, the column-side (right, v) overlap has c theta^2
    a_left = (theta ** 4 - c) / (theta ** 4 + theta ** 2)
    a_right = (theta ** 4 - c) / (theta ** 4 + c * theta ** 2)
    return lam, phi, a_left, a_right


@pytest.mark.parametrize("n,d", [(2000, 1000), (1000, 2000), (1500, 1500)])
def test_white_noise_closed_forms_large(n, d):
    """S = sum theta_i u_i v_i^T + X, X_ij ~ N(0, 1/n): with c = d/n the outlier sits at
    (1+theta^2)(c+theta^2)/theta^2, the bulk edge at (1+sqrt c)^2, d_hat -> theta, the
    overlaps and the Frobenius shrinker -> their Gavish-Donoho / Benaych-Georges-Nadakuditi
    forms.  Singular values come from LAPACK here (the oracle's SVD is pinned above)."""
    rng = np.random.default_rng(n + d)
    c = d / n
    thetas = np.array([4.0, 2.5, 1.6]) * c ** 0.25
    U, _ = np.linalg.qr(rng.standard_normal((n, 3)))
    V, _ = np.linalg.qr(rng.standard_normal((d, 3)))
    S = (U * thetas) @ V.T + rng.standard_normal((n, d)) / math.sqrt(n)
    Uo, sig, Vto = np.linalg.svd(S, full_matrices=False)
    r = oracle.eoptshrink_spectrum(n, d, sig)
    assert r["rank"] == 3
    assert abs(r["lambda_plus"] / (1 + math.sqrt(c)) ** 2 - 1) < 0.03
    for i, th in enumerate(thetas):
        lam, phi, a_left, a_right = _white_closed_form(th, c)
        # the weakest spike's observed location fluctuates by O(d^-1/2 / gap): asymptotic
        # values are compared loosely there, quantities at the observed sigma tightly
        loose = 1.0 if i < 2 else 6.0
        assert abs(sig[i] ** 2 / lam - 1) < 0.03 * loose
        assert abs(r["dhat"][i] / th - 1) < 0.02 * loose
        assert abs(r["a1"][i] - a_left) < 0.01 * loose
        assert abs(r["a2"][i] - a_right) < 0.01 * loose
        assert abs(r["phi"][i] / phi - 1) < 0.03 * loose
        # the overlaps are what they claim to be: squared cosines with the planted vectors
        assert abs((U[:, i] @ Uo[:, i]) ** 2 - r["a1"][i]) < 0.03
        assert abs((V[:, i] @ Vto[i]) ** 2 - r["a2"][i]) < 0.03
        # shrinker evaluated at the observed sigma (removes the outlier-location fluctuation)
        phi_obs = math.sqrt((sig[i] ** 2 - c - 1) ** 2 - 4 * c) / sig[i]
        assert abs(r["phi"][i] / phi_obs - 1) < (0.005 if i < 2 else 0.03)


def test_pr1_reference_block():
    """256 x 128, white noise, spikes at {8,4,2,0.5} x threshold: three detected, the
    sub-threshold one rejected, values near their asymptotic closed forms (c = 1/2)."""
    w = synth.pr1_block(0)
    S = w.blocks[0].double().numpy()
    sig, U, V, _ = oracle.svd(S)
    r = oracle.eoptshrink_spectrum(256, 128, sig)
    assert r["k"] == 11 and r["rank"] == 3
    assert abs(r["lambda_plus"] / 2.914 - 1) < 0.08
    for i, th in enumerate(w.meta["theta"][:3]):
        lam, phi, _, _ = _white_closed_form(th, 0.5)
        assert abs(sig[i] ** 2 / lam - 1) < 0.05
        assert abs(r["dhat"][i] / th - 1) < 0.03
        assert abs(r["phi"][i] / phi - 1) < 0.04
        # identity phi = -T / (sigma T')  (the OptShrink form)
        assert abs(-r["T"][i] / (sig[i] * r["Tp"][i]) - r["phi"][i]) < 1e-12
        assert r["m1"][i] < 0 and r["m2"][i] < 0 and r["T"][i] > 0 and r["Tp"][i] < 0
        assert 0 < r["a1"][i] < 1 and 0 < r["a2"][i] < 1
        assert 0 < r["phi"][i] < sig[i]


# --------------------------------------------------------------------------- #
# Rank selection (Algorithm 2 Step 1; Algorithm 3 else-branch)
# --------------------------------------------------------------------------- #

def test_rank_zero_on_pure_noise_and_cap():
    rng = np.random.default_rng(5)
    for trial in range(12):
        n = int(rng.choice([128, 256, 512]))
        scale = np.exp(rng.uniform(math.log(0.5), math.log(2.0), 128)) if trial % 2 else np.ones(128)
        Z = rng.standard_normal((n, 128)) * scale / math.sqrt(n)
        sig = np.linalg.svd(Z, compute_uv=False)
        assert oracle.eoptshrink_spectrum(n, 128, sig)["rank"] == 0
    # rank never exceeds k: lambda_+ >= lambda_{k+1}
    for trial in range(6):
        lam = np.sort(np.exp(rng.uniform(0, 6, 128)))[::-1]
        assert oracle.eoptshrink_spectrum(256, 128, np.sqrt(lam))["rank"] <= 11


def test_subthreshold_spike_rejected_superthreshold_kept():
    rng = np.random.default_rng(11)
    n, d = 512, 128
    alpha = (d / n) ** 0.25
    u = rng.standard_normal(n); u /= np.linalg.norm(u)
    v = rng.standard_normal(d); v /= np.linalg.norm(v)
    Z = rng.standard_normal((n, d)) / math.sqrt(n)
    assert oracle.eoptshrink_spectrum(n, d, np.linalg.svd(Z + 0.6 * alpha * np.outer(u, v), compute_uv=False))["rank"] == 0
    assert oracle.eoptshrink_spectrum(n, d, np.linalg.svd(Z + 3.0 * alpha * np.outer(u, v), compute_uv=False))["rank"] == 1


# --------------------------------------------------------------------------- #
# TQ stage (Algorithm 1) and the whole pipeline (Algorithm 3)
# --------------------------------------------------------------------------- #

@pytest.mark.parametrize("bits", [1, 2, 3, 4])
def test_tq_stage_distortion_and_ip_shrink(bits):
    """iid Gaussian rows, no low-rank part: relative L2 error of the reconstruction is
    sqrt(D_b) and <y, x_hat>/<y, x> averages 1 - D_b (the MSE quantiser shrinks)."""
    rng = np.random.default_rng(bits)
    n, d = 400, 128
    X = rng.standard_normal((n, d))
    Pi = oracle.rotation(d, 99)
    cen, thr = oracle.codebook(bits, d)
    D = oracle.codebook_distortion(bits, d, cen)
    rho, z, codes = oracle.tq_rows(X, Pi, thr, bits)
    assert np.allclose(rho, np.linalg.norm(X, axis=1), rtol=1e-14)
    assert np.abs(z - (X / rho[:, None]) @ Pi.T).max() < 1e-14
    Xh = oracle.decode(codes, rho, np.zeros((0, n)), np.zeros((0, d)), Pi, cen)
    rel = np.linalg.norm(Xh - X) / np.linalg.norm(X)
    assert abs(rel / math.sqrt(D) - 1) < 0.02
    ratio = np.sum(Xh * X) / np.sum(X * X)
    assert abs(ratio - (1 - D)) < 0.01


def test_brute_force_tiny_block():
    """n = 12, d = 8: every stage against explicit dense numpy / exhaustive search."""
    rng = np.random.default_rng(3)
    n, d, bits = 12, 8, 3
    S = rng.standard_normal((n, d)) * 0.1 + 3.0 * np.outer(rng.standard_normal(n), rng.standard_normal(d))
    Un, sn, Vtn = np.linalg.svd(S, full_matrices=False)
    sig, U, V, _ = oracle.svd(S)
    assert np.allclose(sig, sn, rtol=1e-12)
    r = oracle.eoptshrink_spectrum(n, d, sig, k=2)
    rank = r["rank"]
    assert rank >= 1
    coef = r["phi"][:rank] / sig[:rank]
    R, P = oracle.residual(S, V[:, :rank], coef)
    Shat = (Un[:, :rank] * r["phi"][:rank]) @ Vtn[:rank]
    assert np.abs(R - (S - Shat)).max() < 1e-12
    assert np.abs(P.T @ V[:, :rank].T - Shat).max() < 1e-12
    Pi = oracle.rotation(d, 5)
    cen, thr = oracle.codebook(bits, d)
    rho, z, codes = oracle.tq_rows(R, Pi, thr, bits)
    zb = np.stack([Pi @ (R[t] / np.linalg.norm(R[t])) for t in range(n)])
    assert np.abs(z - zb).max() < 1e-14
    brute = np.argmin(np.abs(zb[:, :, None] - cen[None, None, :]), axis=2)
    assert np.array_equal(codes, brute)
    packed = oracle.pack(codes, bits)
    for t in range(n):  # explicit little-endian bit string
        word = sum(int(codes[t, j]) << (j * bits) for j in range(d))
        assert bytes(packed[t]) == word.to_bytes(d * bits // 8, "little")
    assert np.array_equal(oracle.unpack(packed, d, bits), codes)
    Xh = oracle.decode(codes, rho, P, V[:, :rank].T, Pi, cen)
    assert np.abs(Xh - (Shat + rho[:, None] * (cen[codes] @ Pi))).max() < 1e-12
    Y = rng.standard_normal((3, d))
    assert np.abs(oracle.scores(Xh, Y, 0.25) - 0.25 * Y @ Xh.T).max() < 1e-13
    # zero row: norm 0, reconstructs to the low-rank part only
    R0 = R.copy(); R0[4] = 0
    rho0, z0, codes0 = oracle.tq_rows(R0, Pi, thr, bits)
    assert rho0[4] == 0 and np.all(z0[4] == 0)
    assert np.all(codes0[4] == np.sum(thr < 0))


def test_threshold_tie_takes_lower_index():
    cen, thr = oracle.codebook(2, 128)
    d = 128
    R = np.zeros((1, d)); R[0, 0] = 1.0  # u = e_0, z = Pi[:, 0]
    Pi = np.eye(d)
    # rotation-free case: z_0 = 1 (above all thresholds), the others sit exactly on the middle threshold 0
    _, z, codes = oracle.tq_rows(R, Pi, thr, 2)
    assert codes[0, 0] == 3
    assert thr[1] == 0.0 and np.all(codes[0, 1:] == 1)


def test_pipeline_invariants_on_pr1():
    """Residual has no outliers left and less energy; scale equivariance; row permutation."""
    w = synth.pr1_block(0)
    S = w.blocks[0].double().numpy()
    enc = oracle.encode_blocks(S, 2, 0)
    rank = int(enc["rank"][0])
    assert rank == 3
    V = enc["V"][0, :rank].T
    R, P = oracle.residual(S, V, enc["phi"][0, :rank] / enc["sigma"][0, :rank])
    assert np.linalg.norm(R) < np.linalg.norm(S)
    assert np.allclose(enc["rho"][0], np.linalg.norm(R, axis=1), rtol=1e-13)
    sig_r = np.linalg.svd(R, compute_uv=False)
    assert oracle.eoptshrink_spectrum(256, 128, sig_r)["rank"] == 0
    # the three deflated directions now carry sigma - phi, inside the bulk
    left = enc["sigma"][0, :3] - enc["phi"][0, :3]
    assert np.all(left < math.sqrt(enc["lambda_plus"][0]))
    # scale equivariance
    enc4 = oracle.encode_blocks(4.0 * S, 2, 0)
    assert enc4["rank"][0] == rank and np.array_equal(enc4["packed"], enc["packed"])
    assert np.allclose(enc4["phi"][0, :3], 4 * enc["phi"][0, :3], rtol=1e-12)
    assert np.allclose(enc4["rho"], 4 * enc["rho"], rtol=1e-12)
    # row permutation: spectrum quantities invariant, codes permute with the rows
    perm = np.random.default_rng(0).permutation(256)
    encp = oracle.encode_blocks(S[perm], 2, 0)
    assert encp["rank"][0] == rank
    assert np.allclose(encp["phi"][0, :3], enc["phi"][0, :3], rtol=1e-10)
    diff = np.mean(encp["codes"][0] != enc["codes"][0][perm])
    assert diff < 1e-3
    # reconstruction from stored values is close to the input at the 2-bit distortion level
    X = oracle.decode_stored(enc, 0)
    assert np.linalg.norm(X - S) / np.linalg.norm(S) < np.linalg.norm(R) / np.linalg.norm(S) * 0.36


def test_generator_threshold_white_case():
    lam, alpha = synth.noise_edge_and_threshold(np.ones(128), 1024)
    c = 128 / 1024
    assert abs(lam - (1 + math.sqrt(c)) ** 2) < 1e-9
    assert abs(alpha - c ** 0.25) < 1e-9
