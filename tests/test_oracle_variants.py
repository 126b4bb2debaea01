"""Pins of the oracle's variant helpers: f16 metadata rounding (Section 3.2) and the optional decoder
renormalisation (Section A.3)."""
import numpy as np


def test_f16_rounding_is_ieee_binary16(orc):
    rng = np.random.default_rng(1)
    v = np.concatenate([rng.standard_normal(4000) * np.exp(rng.uniform(-20, 12, 4000)),
                        [0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e9, -1e9, 2.0 ** -24, 2.0 ** -25, 3 * 2.0 ** -25,
                         1.0 + 2.0 ** -11, 1.0 + 3 * 2.0 ** -11, np.inf, -np.inf]]).astype(np.float32)
    with np.errstate(over="ignore"):
        want = v.astype(np.float16).astype(np.float32)  # numpy's own conversion: round to nearest even
    assert np.array_equal(orc.round_f16(v), want)


def test_renormalised_decode_restores_the_row_norm(orc):
    """With r_i / |yhat_i| in place of r_i the decoded row, scaled back by s, has length r_i exactly
    (the rotation is orthonormal, Lemma 1), whereas the plain decoder's length is r_i |yhat_i|."""
    rng = np.random.default_rng(5)
    d_out, d_in, b, K = 7, 512, 128, 64
    W = (rng.standard_normal((d_out, d_in)) * 3).astype(np.float32)
    act = np.exp(rng.standard_normal(d_in)).astype(np.float32)
    s = orc.channel_scales(act, 0.5)
    signs = orc.make_signs(5, d_in)
    sigma, _ = orc.calibrate(W, b, s, signs)
    cb = orc.train_codebook(K, 1 << 12, 2, 20, 1e-5)[0]
    enc = orc.encode(W, b, cb, s, signs, sigma, diagnostics=True)
    adj = orc.renorm_row_norms(enc["packed"], enc["row_norm"], sigma, cb, d_in)
    _, plain = orc.decode(enc["packed"], enc["row_norm"], b, cb, s, signs, sigma, d_in, want_f64=True)
    _, renorm = orc.decode(enc["packed"], adj, b, cb, s, signs, sigma, d_in, want_f64=True)
    len_plain = np.sqrt(((plain * s) ** 2).sum(1))
    len_renorm = np.sqrt(((renorm * s) ** 2).sum(1))
    yhat = cb[enc["idx"]].astype(np.float64) * sigma.astype(np.float64)[None, :, None]
    assert np.allclose(len_plain, enc["row_norm"] * np.sqrt((yhat ** 2).sum((1, 2))), rtol=1e-12)
    assert np.allclose(len_renorm, enc["row_norm"], rtol=2e-7)  # f32 rounding of the factor
    assert not np.allclose(len_plain, enc["row_norm"], rtol=1e-4)  # the plain decoder does not restore it
    # same direction either way
    cos = (plain * renorm).sum(1) / np.sqrt((plain ** 2).sum(1) * (renorm ** 2).sum(1))
    assert np.allclose(cos, 1.0, atol=1e-12)


def test_fused_product_identity(orc):
    """The identity behind the fused decode -> matrix-vector product (Lemma 1: the block Hadamard
    matrix is symmetric and orthonormal): w_hat_i . x = r_i sum_k c_idx_k . (sigma_k xt_k) with
    xt = R_fwd (x / s), checked with the oracle's decoder and forward rotation."""
    rng = np.random.default_rng(8)
    d_out, d_in, b, K = 6, 256, 64, 32
    W = rng.standard_normal((d_out, d_in)).astype(np.float32)
    act = np.exp(rng.standard_normal(d_in)).astype(np.float32)
    s = orc.channel_scales(act, 0.3)
    signs = orc.make_signs(3, d_in)
    sigma, _ = orc.calibrate(W, b, s, signs)
    cb = orc.train_codebook(K, 1 << 12, 1, 20, 1e-5)[0]
    enc = orc.encode(W, b, cb, s, signs, sigma, diagnostics=True)
    _, what = orc.decode(enc["packed"], enc["row_norm"], b, cb, s, signs, sigma, d_in, want_f64=True)
    x = rng.standard_normal(d_in)
    xt = orc.rotate_fwd(x / s.astype(np.float64), signs, b).reshape(-1, 2) * sigma.astype(np.float64)[:, None]
    fused = enc["row_norm"].astype(np.float64) * (cb[enc["idx"]].astype(np.float64) * xt[None]).sum((1, 2))
    assert np.allclose(fused, what @ x, rtol=1e-12, atol=1e-12)
