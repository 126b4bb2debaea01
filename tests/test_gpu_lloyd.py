"""Codebook training on the device (paper Section 3.6) against the oracle's trainer.

Given the same samples the two do the same arithmetic in the same order (exact assignment in double,
cells summed in sample order), so the mean-squared-distance trace, the number of updates and the
final f32 codebook must agree -- the trace to a summation-order tolerance (the oracle adds the
distances in a thread-parallel order), the codebook exactly.
"""
import numpy as np
import pytest
import torch

from conftest import load_golden_codebook

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2605_26339_b200 import binding as q

DEV = "cuda:0"


@pytest.mark.parametrize("K,n,iters", [(1, 4096, 3), (2, 5000, 20), (64, 1 << 14, 25), (256, 1 << 16, 12), (4096, 1 << 15, 4)])
def test_training_on_the_oracles_samples_reproduces_the_oracle(orc, K, n, iters):
    samples = orc.gauss_pairs(9, n)
    ref_cb, ref_mse, ref_iters, ref_trace = orc.train_codebook(K, n, 9, iters, 1e-7, want_trace=True)
    out = q.train_codebook_gpu(K, max_iters=iters, rel_tol=1e-7, samples=torch.from_numpy(samples).to(DEV))
    assert out["iters"] == ref_iters and len(out["trace"]) == len(ref_trace)
    np.testing.assert_allclose(out["trace"], ref_trace, rtol=1e-12)
    assert np.array_equal(out["codebook"], ref_cb)
    assert abs(out["mse"] - ref_mse) <= 1e-12 * ref_mse
    if K == 1:  # one cell: its codeword is the sample mean, the distortion the total variance
        assert np.allclose(out["codebook"][0], samples.mean(0), atol=1e-7)


def test_assignment_and_centroids_of_one_iteration(orc):
    """One update from a known codebook: the new codewords are the means of the oracle's cells."""
    n, K = 20000, 32
    samples = orc.gauss_pairs(3, n)
    out = q.train_codebook_gpu(K, max_iters=1, rel_tol=0.0, samples=torch.from_numpy(samples).to(DEV))
    cb0 = np.sqrt(2.0) * samples[:K]
    assign, mse0 = orc.lloyd_assign(samples, cb0)
    assert abs(out["trace"][0] - mse0) <= 1e-12 * mse0
    want = cb0.copy()
    for c in range(K):
        if (assign == c).any():
            want[c] = samples[assign == c].mean(0)
    order = np.lexsort((np.arctan2(want[:, 1], want[:, 0]), (want ** 2).sum(1)))
    assert np.allclose(out["codebook"], want[order].astype(np.float32), atol=1e-6)


def test_device_generated_samples_give_the_golden_codebook_quality(orc):
    """Without a sample array the device draws the counter-based Gaussian stream itself (its log / sin /
    cos may differ from the host's in the last bit, so codewords are compared to a tolerance) and the
    trained codebook has the distortion of the oracle-trained golden one."""
    K = 256
    hdr_mse = orc.codebook_mse(load_golden_codebook(K), 1 << 16, 1234)
    out = q.train_codebook_gpu(K, 1 << 20, 0, 100, 1e-6)
    assert abs(orc.codebook_mse(out["codebook"], 1 << 16, 1234) - hdr_mse) < 0.01 * hdr_mse
    host_cb, host_mse = q.train_codebook(K, 1 << 20, 0, 100, 1e-6)
    assert abs(out["mse"] - host_mse) < 1e-6 * host_mse
    assert np.abs(out["codebook"] - host_cb).max() < 1e-4
    print(f"LLOYD K={K}: device {out['seconds']:.3f} s, {out['iters']} updates")
    again = q.train_codebook_gpu(K, 1 << 20, 0, 100, 1e-6)
    assert np.array_equal(again["codebook"], out["codebook"])  # reproducible run to run


def test_codebook_fitted_to_a_matrix_beats_the_gaussian_one_on_it(orc):
    """Per-matrix codebook (Lloyd on the matrix's own rotated, scaled pairs): its quantisation error on
    those pairs is not above the Gaussian-trained codebook's, and the device trainer's result on the
    pairs equals the oracle trainer's."""
    from paper_2605_26339_b200.model_codec import fit_codebook
    g = torch.Generator().manual_seed(12)
    d_out, d_in, K = 512, 1024, 64
    # light-tailed rows (uniform entries): after a block-32 rotation the pairs are visibly non-Gaussian
    W = ((torch.rand((d_out, d_in), generator=g) - 0.5) * torch.exp(0.5 * torch.randn((d_out, 1), generator=g))).to(DEV)
    fit = fit_codebook(W, None, 0.0, 2, K, n_pairs=1 << 16, max_iters=40, rel_tol=1e-7)
    assert fit["codebook"].shape == (K, 2) and np.isfinite(fit["codebook"]).all()
    # the same pairs through the oracle: same codebook
    rows = (np.arange(fit["rows"]) * d_out) // fit["rows"]
    signs = q.make_signs(q.DEFAULT_SIGN_SEED, d_in)
    Wh = W.cpu().numpy()
    y = np.stack([orc.front_row(Wh[r], 2, None, signs)[0] for r in rows])
    z = (y.reshape(len(rows), d_in // 2, 2) / fit["sigma"].cpu().numpy()[None, :, None]).reshape(-1, 2)[: 1 << 16]
    ref_cb, ref_mse, _, _ = orc.train_codebook_on(z.astype(np.float64), K, 40, 1e-7)
    assert np.array_equal(fit["codebook"], ref_cb)
    gauss = load_golden_codebook(K)
    _, mse_gauss = orc.lloyd_assign(z.astype(np.float64), gauss.astype(np.float64))
    assert fit["mse"] < mse_gauss
