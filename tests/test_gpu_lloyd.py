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
