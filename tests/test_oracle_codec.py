"""Pins of the oracle's codebook trainer, nearest-codeword search, encoder,
decoder and distortion sums.  Expected values: the paper's identities and
printed figures, textbook closed forms (scalar Lloyd-Max, Zador-Gersho),
library routines (scipy cKDTree, numpy), and exhaustive evaluation."""
import numpy as np
import pytest
import torch
from scipy.spatial import cKDTree
from scipy.special import erf

from conftest import golden_header, load_golden_codebook


# ----------------------------------------------------------------------------- samples
def test_gauss_pairs_statistics(orc):
    """Unit circular Gaussian (Section 3.6 equation): zero mean, identity covariance,
    Rayleigh modulus with E|z| = sqrt(pi/2) (Section 3.4), uniform phase."""
    z = orc.gauss_pairs(0, 1 << 18)
    n = z.shape[0]
    assert np.all(np.abs(z.mean(0)) < 5 / np.sqrt(n))
    cov = z.T @ z / n
    np.testing.assert_allclose(cov, np.eye(2), atol=5 * np.sqrt(2.0 / n))
    amp = np.hypot(z[:, 0], z[:, 1])
    assert abs(amp.mean() - np.sqrt(np.pi / 2)) < 5 * 0.655 / np.sqrt(n)
    assert abs((amp**2).mean() - 2.0) < 5 * 2.0 / np.sqrt(n)
    # Rayleigh CDF at a few radii
    for r0 in (0.5, 1.0, 2.0, 3.0):
        p = 1 - np.exp(-r0 * r0 / 2)
        assert abs((amp < r0).mean() - p) < 5 * np.sqrt(p * (1 - p) / n)
    ph = np.arctan2(z[:, 1], z[:, 0])
    hist = np.histogram(ph, bins=16, range=(-np.pi, np.pi))[0] / n
    assert np.all(np.abs(hist - 1 / 16) < 5 * np.sqrt(1 / 16 / n))
    # streams: another seed is another stream, same seed repeats, prefix property
    assert not np.array_equal(orc.gauss_pairs(1, 64), z[:64])
    assert np.array_equal(orc.gauss_pairs(0, 64), z[:64])


# ----------------------------------------------------------------------------- Lloyd
def test_lloyd_k1_is_the_mean(orc):
    cb, mse, iters = orc.train_codebook(1, 1 << 14, 3, 10, 0.0)
    z = orc.gauss_pairs(3, 1 << 14)
    np.testing.assert_allclose(cb[0], z.mean(0), atol=1e-7)
    assert abs(mse - ((z - cb[0].astype(np.float64)) ** 2).sum(1).mean()) < 1e-12
    assert abs(mse - 2.0) < 0.05  # E|z|^2 = 2


def test_lloyd_fixed_point_conditions(orc):
    """Run to an exact fixed point (rel_tol = 0): nearest-neighbour and centroid conditions,
    monotone training MSE, and the centroid identity E|Q|^2 = E|z|^2 - D (the 2-D form of the
    argument in the proof of Corollary 2)."""
    K, n = 16, 1 << 14
    cb, mse, iters, trace = orc.train_codebook(K, n, 5, 2000, 0.0, want_trace=True)
    assert iters < 2000  # converged, not cut off
    assert np.all(np.diff(trace) <= 1e-15)  # Lloyd never increases the training MSE
    z = orc.gauss_pairs(5, n)
    assign, mse2 = orc.lloyd_assign(z, cb.astype(np.float64))
    assert abs(mse2 - mse) < 1e-15
    # nearest-neighbour condition through an independent library routine
    _, nn = cKDTree(cb.astype(np.float64)).query(z)
    assert np.array_equal(nn, assign)
    # centroid condition (codebook is stored as f32)
    cnt = np.bincount(assign, minlength=K)
    cen = np.stack([np.bincount(assign, z[:, d], K) / cnt for d in (0, 1)], 1)
    np.testing.assert_allclose(cb, cen, atol=2e-7)
    p = cnt / n
    lhs = (p * (cb.astype(np.float64) ** 2).sum(1)).sum()
    assert abs(lhs - ((z**2).sum(1).mean() - mse)) < 1e-6
    # sorted by radius
    assert np.all(np.diff((cb.astype(np.float64) ** 2).sum(1)) >= 0)


def test_lloyd_init_is_scaled_samples(orc):
    """max_iters = 0: the codebook is sqrt(2) x the first K samples (sorted by radius)."""
    K = 32
    cb, _, iters = orc.train_codebook(K, 1 << 10, 8, 0, 0.0)
    z = orc.gauss_pairs(8, K) * np.sqrt(2.0)
    order = np.argsort((z**2).sum(1), kind="stable")
    assert iters == 0
    np.testing.assert_allclose(cb, z[order], rtol=1e-7)


def _scalar_lloyd_max_mse(levels: int) -> float:
    """Textbook scalar Lloyd-Max quantiser for N(0,1), by closed-form Gaussian cell moments."""
    phi = lambda t: np.exp(-0.5 * t * t) / np.sqrt(2 * np.pi)
    Phi = lambda t: 0.5 * (1 + erf(t / np.sqrt(2)))
    x = np.linspace(-2.5, 2.5, levels)
    for _ in range(20000):
        t = np.concatenate([[-np.inf], 0.5 * (x[1:] + x[:-1]), [np.inf]])
        mass = Phi(t[1:]) - Phi(t[:-1])
        new = (phi(t[:-1]) - phi(t[1:])) / mass
        if np.max(np.abs(new - x)) < 1e-13:
            x = new
            break
        x = new
    return 1.0 - (mass * x * x).sum()  # centroid identity: D = E U^2 - E Q^2


def test_scalar_lloyd_max_textbook_values():
    # Max (1960), Table I: 4 levels 0.1175, 8 levels 0.03454
    assert abs(_scalar_lloyd_max_mse(4) - 0.1175) < 1e-4
    assert abs(_scalar_lloyd_max_mse(8) - 0.03454) < 1e-5


@pytest.mark.parametrize("K", [64, 256, 1024, 2048, 4096])
def test_golden_codebook_quality(orc, K):
    """The oracle-trained codebooks stored under tests/golden: training MSE as recorded,
    fresh-sample Monte-Carlo MSE close to it, better than the product of two scalar Lloyd-Max
    quantisers, inside the high-rate band D_B ~ 2 G(2) |f|_{1/2} / K = 4.03 / K (Zador-Gersho;
    the paper's consequence (C1) quotes the 2 G(2) 2^-B scaling), halving per extra bit."""
    cb = load_golden_codebook(K)
    hdr = golden_header(K)
    assert np.all(np.diff((cb.astype(np.float64) ** 2).sum(1)) >= 0)
    assert len({tuple(c) for c in cb.tolist()}) == K  # distinct codewords
    n = 1 << 17 if K > 1024 else 1 << 18
    fresh = orc.codebook_mse(cb, n, 77)
    train = float(hdr["train_mse"])
    # the training MSE is optimistic by O(K / n_samples) (fewer samples per cell at larger K)
    assert 0 <= fresh - train < (0.02 + 16 * K / (1 << 20)) * train
    L = int(round(np.sqrt(K)))
    if L * L == K:
        assert fresh < 2 * _scalar_lloyd_max_mse(L)
    zador = 2 * (5 / (36 * np.sqrt(3))) * 8 * np.pi / K
    assert 0.93 * zador < fresh < 1.12 * zador
    # centroid property in aggregate: the probability-weighted mean of the codewords is E z = 0
    z = orc.gauss_pairs(78, 1 << 16)
    assign, _ = orc.lloyd_assign(z, cb.astype(np.float64))
    p = np.bincount(assign, minlength=K) / z.shape[0]
    assert np.abs((p[:, None] * cb.astype(np.float64)).sum(0)).max() < 0.02


def test_golden_codebook_halving_per_bit(orc):
    d = {K: float(golden_header(K)["train_mse"]) for K in (64, 128, 256, 1024, 2048, 4096)}
    for a, b in ((64, 128), (128, 256), (1024, 2048), (2048, 4096)):
        assert 0.48 < d[b] / d[a] < 0.54


def test_golden_codebook_is_what_the_oracle_trains(orc):
    """The stored file is reproducible from the committed script (checked at K = 64)."""
    cb, mse, iters = orc.train_codebook(64, 1 << 20, 0, 100, 1e-6)
    assert np.array_equal(cb, load_golden_codebook(64))


# ----------------------------------------------------------------------------- search
def test_nearest_against_kdtree_and_exhaustive(orc):
    cb = load_golden_codebook(2048)
    rng = np.random.default_rng(1)
    z = (rng.standard_normal((20000, 2)) * 1.3).astype(np.float32)
    idx, d1, d2 = orc.nearest(z, cb)
    dist, nn = cKDTree(cb.astype(np.float64)).query(z.astype(np.float64), k=2)
    np.testing.assert_allclose(d1, dist[:, 0] ** 2, rtol=1e-12, atol=1e-300)
    np.testing.assert_allclose(d2, dist[:, 1] ** 2, rtol=1e-12, atol=1e-300)
    clear = (d2 - d1) > 1e-12 * d2
    assert np.array_equal(idx[clear], nn[clear, 0])
    assert np.all(d1 <= d2)


def test_nearest_tiny_cases(orc):
    cb = np.array([[0, 0], [1, 0], [0, 1], [1, 1]], np.float32)
    idx, d1, d2 = orc.nearest(np.array([[0.2, 0.1], [0.9, 0.2], [0.5, 0.5], [0.4, 0.9], [5, 5]]), cb)
    assert idx.tolist() == [0, 1, 0, 2, 3]  # exact 4-way tie -> lowest index
    assert d1[2] == d2[2] == 0.5
    idx, d1, d2 = orc.nearest(np.array([[3.0, -4.0]]), np.array([[0, 0]], np.float32))  # K = 1
    assert idx[0] == 0 and d1[0] == 25.0 and np.isinf(d2[0])


# ----------------------------------------------------------------------------- codec
def _problem(orc, d_out, d_in, b, K, dtype="f32", alpha=0.5, seed=0, gaussian=False):
    rng = np.random.default_rng(seed)
    if gaussian:
        W = rng.standard_normal((d_out, d_in)).astype(np.float32)
    else:
        W = (rng.standard_t(5, (d_out, d_in)) * np.exp(0.5 * rng.standard_normal((d_out, 1)))).astype(np.float32)
    if dtype == "bf16":
        W = torch.from_numpy(W).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    act = np.exp(rng.standard_normal(d_in)).astype(np.float32)
    s = orc.channel_scales(act, alpha) if alpha else None
    signs = orc.make_signs(0x51A5, d_in)
    sigma, rc = orc.calibrate(W, b, s, signs)
    assert rc == 0
    return W, act, s, signs, sigma, load_golden_codebook(K)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_encode_is_rotated_nearest_codeword(orc, dtype):
    """decode(encode(x)) in the rotated, sigma-scaled domain is the nearest codeword, and
    |u - u~|^2 = sum_k sigma_k^2 |z_k - c|^2 (Section A.3 equation)."""
    d_out, d_in, b, K = 24, 512, 128, 256
    W, act, s, signs, sigma, cb = _problem(orc, d_out, d_in, b, K, dtype, seed=2)
    enc = orc.encode(W, b, cb, s, signs, sigma, diagnostics=True)
    assert enc["status"] == 0
    what, w64 = orc.decode(enc["packed"], enc["row_norm"], b, cb, s, signs, sigma, d_in, want_f64=True)
    Wf = orc.bf16_to_f32(W).astype(np.float64) if dtype == "bf16" else W.astype(np.float64)
    sd = np.ones(d_in) if s is None else s.astype(np.float64)
    for i in range(d_out):
        # indices: exhaustive search on the definition-path z agrees wherever the gap is clear
        y64, r64, _ = orc.front_row_def(W[i], b, s, signs)
        z64 = y64.reshape(-1, 2) / sigma.astype(np.float64)[:, None]
        np.testing.assert_allclose(enc["z"][i], z64, rtol=0, atol=2e-5 * np.abs(z64).max())
        idx_def, d1, d2 = orc.nearest(z64, cb)
        clear = (d2 - d1) > 1e-3 * d2
        assert clear.mean() > 0.95
        assert np.array_equal(enc["idx"][i][clear], idx_def[clear])
        # packed stream holds exactly those indices
        assert np.array_equal(orc.unpack_row(enc["packed"][i], d_in // 2, 8), enc["idx"][i])
        # decoded direction in the rotated domain = chosen codeword x sigma
        u_tilde = w64[i] * sd / float(enc["row_norm"][i])
        y_hat = orc.rotate_fwd(u_tilde, signs, b).reshape(-1, 2)
        c = cb[enc["idx"][i]].astype(np.float64) * sigma.astype(np.float64)[:, None]
        np.testing.assert_allclose(y_hat, c, atol=1e-12)
        # error accounting identity
        u = Wf[i] * sd / r64
        lhs = ((u - u_tilde) ** 2).sum()
        rhs = ((sigma.astype(np.float64) ** 2) * ((z64 - cb[enc["idx"][i]].astype(np.float64)) ** 2).sum(1)).sum()
        assert abs(lhs - rhs) < 1e-6 * rhs
    # bf16 output is the one-rounding image of the double result
    assert np.array_equal(what, orc.f64_to_bf16(w64))


def test_encode_gap_report_and_tie_rule(orc):
    d_out, d_in, b, K = 8, 256, 64, 64
    W, act, s, signs, sigma, cb = _problem(orc, d_out, d_in, b, K, seed=4)
    enc = orc.encode(W, b, cb, s, signs, sigma, diagnostics=True)
    z = enc["z"].astype(np.float64).reshape(-1, 2)
    d = ((z[:, None, :] - cb.astype(np.float64)[None]) ** 2).sum(2)  # numpy exhaustive
    order = np.argsort(d, axis=1, kind="stable")
    assert np.array_equal(enc["idx"].ravel(), order[:, 0])
    np.testing.assert_allclose(enc["d2_best"].ravel(), np.take_along_axis(d, order[:, :1], 1)[:, 0], rtol=1e-13)
    np.testing.assert_allclose(enc["d2_second"].ravel(), np.take_along_axis(d, order[:, 1:2], 1)[:, 0], rtol=1e-13)


def test_encode_zero_and_nonfinite_rows(orc):
    d_in, b, K = 128, 64, 64
    cb = load_golden_codebook(K)
    signs = orc.make_signs(1, d_in)
    sigma = np.full(d_in // 2, 1 / np.sqrt(d_in), np.float32)
    W = np.random.default_rng(0).standard_normal((4, d_in)).astype(np.float32)
    W[1] = 0
    enc = orc.encode(W, b, cb, None, signs, sigma, diagnostics=True)
    origin = orc.nearest(np.zeros((1, 2)), cb)[0][0]
    assert enc["status"] == 0 and enc["row_norm"][1] == 0
    assert np.all(enc["idx"][1] == origin)  # zero row: every pair is the origin's codeword
    what = orc.decode(enc["packed"], enc["row_norm"], b, cb, None, signs, sigma, d_in)
    assert not orc.bf16_to_f32(what[1]).any()  # and decodes to zeros
    W[2, 7] = np.inf
    enc = orc.encode(W, b, cb, None, signs, sigma)
    assert enc["status"] == orc.ORC_ERR_NONFINITE


def test_packed_row_stride_and_padding(orc):
    d_in, b, K = 64, 32, 128  # 32 pairs x 7 bits = 224 bits = 28 bytes
    cb = load_golden_codebook(K)
    signs = orc.make_signs(1, d_in)
    sigma = np.full(d_in // 2, 1 / np.sqrt(d_in), np.float32)
    W = np.random.default_rng(3).standard_normal((5, d_in)).astype(np.float32)
    a = orc.encode(W, b, cb, None, signs, sigma)
    c = orc.encode(W, b, cb, None, signs, sigma, packed_row_stride=48)
    assert a["packed"].shape == (5, 28) and c["packed"].shape == (5, 48)
    assert np.array_equal(c["packed"][:, :28], a["packed"]) and not c["packed"][:, 28:].any()


def test_gaussian_rows_weight_error_matches_codebook_mse(orc):
    """Equation (weight-mse) with Gaussian rows and no channel scaling: rho_w^2 ~ D_B / 2.
    The paper's measured rho_w = 0.033 at B = 11 (Table "layer-diag") sits at sqrt(D_2048/2)."""
    d_out, d_in, b = 96, 1024, 128
    for K, tol in ((256, 0.05), (2048, 0.05)):
        W, act, s, signs, sigma, cb = _problem(orc, d_out, d_in, b, K, alpha=0.0, seed=6, gaussian=True)
        enc = orc.encode(W, b, cb, None, signs, sigma)
        what = orc.decode(enc["packed"], enc["row_norm"], b, cb, None, signs, sigma, d_in)
        s4 = orc.distortion(W, what, None)
        D = float(golden_header(K)["train_mse"])
        bf16_floor = (2.0**-9) ** 2 / 3  # rounding the output to bf16 adds ~ u^2/3 relative
        rho2 = s4[0] / s4[1] - bf16_floor
        assert abs(rho2 - D / 2) < tol * D / 2, (K, rho2, D / 2)
    assert abs(np.sqrt(float(golden_header(2048)["train_mse"]) / 2) - 0.033) < 0.002


def test_distortion_sums(orc):
    """Corollary 4 (diagonal M_x): sum_ij r_j^2 dW_ij^2 equals |X dW^T|_F^2 / n when the
    activations have diagonal second moment; checked with explicit X = diag(r) (n = d_in)."""
    rng = np.random.default_rng(12)
    d_out, d_in = 7, 32
    W = rng.standard_normal((d_out, d_in)).astype(np.float32)
    What = torch.from_numpy(W + 0.05 * rng.standard_normal((d_out, d_in)).astype(np.float32)).to(torch.bfloat16)
    bits = What.view(torch.int16).numpy().view(np.uint16)
    r = np.exp(rng.standard_normal(d_in)).astype(np.float32)
    s4 = orc.distortion(W, bits, r)
    dW = W.astype(np.float64) - What.to(torch.float64).numpy()
    X = np.diag(r.astype(np.float64)) * np.sqrt(d_in)  # X^T X / n = diag(r^2)
    assert abs(s4[0] - np.linalg.norm(dW) ** 2) < 1e-12 * s4[0]
    assert abs(s4[1] - np.linalg.norm(W.astype(np.float64)) ** 2) < 1e-12 * s4[1]
    assert abs(s4[2] - np.linalg.norm(X @ dW.T) ** 2 / d_in) < 1e-12 * s4[2]
    assert abs(s4[3] - np.linalg.norm(X @ W.astype(np.float64).T) ** 2 / d_in) < 1e-12 * s4[3]
    s4n = orc.distortion(W, bits, None)
    assert s4n[0] == s4n[2] and s4n[1] == s4n[3]


def test_channel_scaling_is_undone_by_decode(orc):
    """Section B.2: W_hat = Quantize(W D_s) D_s^-1.  Encoding W with scales s must equal
    encoding the pre-scaled matrix W D_s without scales, then dividing the columns by s."""
    d_out, d_in, b, K = 6, 256, 128, 256
    W, act, s, signs, sigma, cb = _problem(orc, d_out, d_in, b, K, alpha=0.5, seed=8)
    s2 = 2.0 ** np.round(np.log2(s))  # power-of-two scales keep W D_s exact in f32
    s2 = s2.astype(np.float32)
    a = orc.encode(W, b, cb, s2, signs, sigma)
    c = orc.encode((W * s2).astype(np.float32), b, cb, None, signs, sigma)
    assert np.array_equal(a["packed"], c["packed"]) and np.array_equal(a["row_norm"], c["row_norm"])
    _, wa = orc.decode(a["packed"], a["row_norm"], b, cb, s2, signs, sigma, d_in, want_f64=True)
    _, wc = orc.decode(c["packed"], c["row_norm"], b, cb, None, signs, sigma, d_in, want_f64=True)
    np.testing.assert_allclose(wa, wc / s2.astype(np.float64), rtol=1e-15)
