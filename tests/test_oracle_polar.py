"""Pins of the oracle's polar baseline codec (paper Section 3.5, the pairwise distortion theorem's
corollary for the Rayleigh / uniform-phase source and the remark on the cut-off R_max = 8).

Each check compares the oracle with something it does not compute itself: closed forms of the unit
Rayleigh law, scipy quadrature and optimisation, numpy brute force, the corollary's formula on
Monte-Carlo samples.
"""
import numpy as np
import pytest
from scipy import integrate, optimize


def _pdf(r):
    return r * np.exp(-0.5 * r * r)


def _cell_bounds(levels):
    lv = np.asarray(levels, np.float64)
    mid = 0.5 * (lv[1:] + lv[:-1])
    return np.concatenate([[0.0], mid]), np.concatenate([mid, [8.0]])


def test_single_level_is_the_rayleigh_mean(orc):
    """N_a = 1: the centroid of the whole law is E U = sqrt(pi/2) and C_LM = Var U = 2 - pi/2."""
    lv, c = orc.rayleigh_lloyd_max(1)
    assert lv[0] == np.float32(np.sqrt(np.pi / 2))
    assert abs(c - (2 - np.pi / 2)) < 1e-9


@pytest.mark.parametrize("n", [2, 4, 32])
def test_levels_satisfy_the_lloyd_max_conditions(orc, n):
    """Every level is the centroid of its cell (cells bounded by midpoints), checked with scipy's
    quadrature; the reported distortion is the integral of (r - Q(r))^2 f(r); and the centroid
    identity of the corollary's proof holds: E[U Q(U)] = E[Q(U)^2] = 2 - C_LM."""
    lv, c = orc.rayleigh_lloyd_max(n)
    assert np.all(np.diff(lv) > 0) and lv[0] > 0
    lo, hi = _cell_bounds(lv)
    D = M = Q2 = 0.0
    for j in range(n):
        m0 = integrate.quad(_pdf, lo[j], hi[j], epsabs=1e-13, epsrel=1e-13)[0]
        m1 = integrate.quad(lambda r: r * _pdf(r), lo[j], hi[j], epsabs=1e-13, epsrel=1e-13)[0]
        assert abs(m1 / m0 - lv[j]) < 2e-7 * max(1.0, lv[j])  # f32 rounding of the level
        D += integrate.quad(lambda r: (r - float(lv[j])) ** 2 * _pdf(r), lo[j], hi[j], epsabs=1e-13, epsrel=1e-13)[0]
        M += float(lv[j]) * m1
        Q2 += float(lv[j]) ** 2 * m0
    assert abs(D - c) < 1e-9
    assert abs(M - Q2) < 1e-6 and abs((2 - c) - M) < 1e-6
    assert abs(orc.rayleigh_distortion(lv) - c) < 1e-12


@pytest.mark.parametrize("n", [2, 3])
def test_small_quantisers_match_a_direct_minimisation(orc, n):
    """The Lloyd fixed point is the minimiser of the distortion: scipy's optimiser over the levels,
    started elsewhere, finds the same levels."""
    lv, c = orc.rayleigh_lloyd_max(n)

    def dist(x):
        x = np.sort(np.abs(x))
        lo, hi = _cell_bounds(x)
        return sum(integrate.quad(lambda r: (r - x[j]) ** 2 * _pdf(r), lo[j], hi[j])[0] for j in range(n))

    res = optimize.minimize(dist, np.linspace(0.5, 2.5, n), method="Nelder-Mead", options=dict(xatol=1e-7, fatol=1e-13))
    assert np.allclose(np.sort(res.x), lv, atol=2e-5)
    assert abs(res.fun - c) < 1e-8


def test_polar_codebook_layout(orc):
    """index = (phase << Ba) | amplitude; bin centres at odd multiples of pi / N_p."""
    Ba, Bp = 3, 4
    lv, _ = orc.rayleigh_lloyd_max(1 << Ba)
    cb = orc.polar_codebook(lv, Ba, Bp).astype(np.float64)
    assert cb.shape == (128, 2)
    rad = np.hypot(cb[:, 0], cb[:, 1]).reshape(16, 8)
    ang = np.mod(np.arctan2(cb[:, 1], cb[:, 0]), 2 * np.pi).reshape(16, 8)
    assert np.allclose(rad, lv[None, :], rtol=2e-7)
    assert np.allclose(ang, ((2 * np.arange(16) + 1) * np.pi / 16)[:, None], atol=1e-6)


def test_polar_quantiser_against_numpy_brute_force(orc):
    Ba, Bp = 5, 6
    lv, _ = orc.rayleigh_lloyd_max(1 << Ba)
    z = orc.gauss_pairs(11, 4000) * 1.3
    idx, ma, mp = orc.polar_quantize(z, lv, Ba, Bp)
    r = np.hypot(z[:, 0], z[:, 1])
    a_ref = np.abs(r[:, None] - lv.astype(np.float64)[None, :]).argmin(1)
    theta = np.mod(np.arctan2(z[:, 1], z[:, 0]), 2 * np.pi)
    p_ref = np.floor(theta / (2 * np.pi / 64)).astype(int)
    clear = (ma > 1e-9) & (mp > 1e-9)
    assert clear.mean() > 0.999
    assert np.array_equal(idx[clear] & 31, a_ref[clear]) and np.array_equal(idx[clear] >> 5, p_ref[clear])
    # a point on a bin centre sits half a bin from both boundaries; the origin goes to bin 0, level 0
    h = np.pi / 64
    centres = np.stack([np.cos((2 * np.arange(64) + 1) * h), np.sin((2 * np.arange(64) + 1) * h)], 1) * float(lv[7])
    ic, mac, mpc = orc.polar_quantize(centres, lv, Ba, Bp)
    assert np.array_equal(ic >> 5, np.arange(64)) and np.all(ic & 31 == 7) and np.allclose(mpc, h, atol=1e-9)
    i0, _, mp0 = orc.polar_quantize(np.array([[0.0, 0.0], [-0.0, -0.0]]), lv, Ba, Bp)
    assert np.all(i0 == 0) and np.all(mp0 == np.pi)
    # just below the positive x axis: the last bin, not bin N_p
    il, _, _ = orc.polar_quantize(np.array([[1.0, -1e-18]]), lv, Ba, Bp)
    assert il[0] >> 5 == 63


@pytest.mark.parametrize("Ba,Bp", [(5, 6), (3, 4), (0, 3), (4, 0)])
def test_corollary_closed_form_on_monte_carlo_samples(orc, Ba, Bp):
    """E|z - zhat|^2 = C_LM + 2 (2 - C_LM) eta(N_p), eta = 1 - sin(pi/N_p) / (pi/N_p), for the unit
    circular Gaussian source; and the corollary's upper bound with pi^2 / (3 N_p^2)."""
    n = 1 << 17
    lv, c = orc.rayleigh_lloyd_max(1 << Ba)
    cb = orc.polar_codebook(lv, Ba, Bp).astype(np.float64)
    z = orc.gauss_pairs(5, n)
    idx, _, _ = orc.polar_quantize(z, lv, Ba, Bp)
    err = ((z - cb[idx]) ** 2).sum(1)
    Np = 1 << Bp
    eta = 1 - np.sin(np.pi / Np) / (np.pi / Np)
    want = c + 2 * (2 - c) * eta
    assert abs(err.mean() - want) < 4 * err.std() / np.sqrt(n) + 1e-6
    assert want <= c + (2 - c) * np.pi ** 2 / (3 * Np ** 2) + 1e-12


def test_polar_encoder_is_front_half_plus_quantiser(orc):
    """orc_encode_polar = the common front half (z as in the 2-D encoder) followed by the polar
    quantiser per pair; decoding its stream with the product table reproduces the polar
    reconstruction in the rotated, scaled domain."""
    rng = np.random.default_rng(3)
    d_out, d_in, b, Ba, Bp = 9, 256, 64, 4, 5
    W = rng.standard_normal((d_out, d_in)).astype(np.float32)
    signs = orc.make_signs(77, d_in)
    sigma, _ = orc.calibrate(W, b, None, signs)
    lv, _ = orc.rayleigh_lloyd_max(1 << Ba)
    cb = orc.polar_codebook(lv, Ba, Bp)
    enc = orc.encode_polar(W, b, lv, Ba, Bp, None, signs, sigma, diagnostics=True)
    ref = orc.encode(W, b, cb, None, signs, sigma, diagnostics=True)  # same front half
    assert np.array_equal(enc["z"], ref["z"]) and np.array_equal(enc["row_norm"], ref["row_norm"])
    idx, ma, mp = orc.polar_quantize(enc["z"].reshape(-1, 2), lv, Ba, Bp)
    assert np.array_equal(idx.reshape(d_out, -1), enc["idx"])
    got = np.stack([orc.unpack_row(r, d_in // 2, Ba + Bp) for r in enc["packed"]])
    assert np.array_equal(got, enc["idx"])
    # the polar rule is not the nearest-neighbour rule of the product table: some pairs differ
    assert (enc["idx"] != ref["idx"]).any()
    # decode: rotating the decoded unit direction forward gives codeword * sigma
    what, w64 = orc.decode(enc["packed"], enc["row_norm"], b, cb, None, signs, sigma, d_in, want_f64=True)
    for i in range(d_out):
        u = w64[i] / float(enc["row_norm"][i])
        y = orc.rotate_fwd(u, signs, b).reshape(-1, 2)
        assert np.allclose(y, cb[enc["idx"][i]].astype(np.float64) * sigma.astype(np.float64)[:, None], atol=1e-12)
