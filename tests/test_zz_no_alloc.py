"""qamw_calibrate_static: calibration for callers that cannot allocate device memory.

An embedding application that owns the device heap (a server with a fixed memory plan, a plug-in
running inside someone else's stream) cannot hand qamw_calibrate a scratch buffer.  The static
variant keeps its partial sums in an array compiled into the library.  Here it is called through
the C ABI twice in a row, on two different shapes, so that the second call runs on scratch that
still holds the first call's partial sums; each result must equal what qamw_calibrate computes
with a caller-provided workspace, within the calibration tolerance of the parity tests.
This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
"""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2605_26339_b200 import binding as q

DEV = "cuda:0"


def _problem(d_out, d_in, dtype, seed):
    g = torch.Generator().manual_seed(seed)
    W = (torch.randn((d_out, d_in), generator=g) * torch.exp(0.5 * torch.randn((d_out, 1), generator=g))).to(dtype)
    act = torch.exp(torch.randn(d_in, generator=g)).numpy().astype(np.float32)
    s = torch.from_numpy(q.channel_scales(act, 0.3)).to(DEV)
    signs = torch.from_numpy(q.make_signs(q.DEFAULT_SIGN_SEED, d_in)).to(DEV)
    return W.to(DEV), s, signs


def _both(d_out, d_in, block, dtype, seed):
    W, s, signs = _problem(d_out, d_in, dtype, seed)
    p = q.make_params(W, d_out, d_in, block, 256)
    assert q.calibrate_workspace_bytes(p) <= q.STATIC_SCRATCH_BYTES
    ws = torch.empty(q.calibrate_workspace_bytes(p), dtype=torch.uint8, device=DEV)
    ref = torch.empty(d_in // 2, dtype=torch.float32, device=DEV)
    st_ref = torch.zeros(1, dtype=torch.int32, device=DEV)
    q.calibrate(W, p, s, signs, ref, ws, st_ref)
    got = torch.full((d_in // 2,), float("nan"), dtype=torch.float32, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    q.calibrate_static(W, p, s, signs, got, st)
    torch.cuda.synchronize()
    assert int(st.cpu()[0]) == int(st_ref.cpu()[0]) == 0
    return got.cpu().numpy(), ref.cpu().numpy()


def test_static_scratch_matches_workspace_variant_twice_in_a_row():
    # first call: a wide matrix that fills a large part of the built-in scratch
    got, ref = _both(1500, 4096, 128, torch.bfloat16, 1)
    np.testing.assert_allclose(got, ref, rtol=1e-5)
    assert np.all(np.isfinite(got)) and np.all(got > 0)
    # second call, straight after, on a smaller shape: the scratch still holds the first call's sums
    got2, ref2 = _both(700, 1024, 64, torch.float32, 2)
    np.testing.assert_allclose(got2, ref2, rtol=1e-5)
    # and the first shape again
    got3, ref3 = _both(1500, 4096, 128, torch.bfloat16, 1)
    np.testing.assert_allclose(got3, ref3, rtol=1e-5)
    assert np.array_equal(got3, got)
    # the call itself takes no device memory: free memory is the same before and after a call whose
    # tensors all exist already
    W, s, signs = _problem(1500, 4096, torch.bfloat16, 1)
    p = q.make_params(W, 1500, 4096, 128, 256)
    out = torch.empty(2048, dtype=torch.float32, device=DEV)
    q.calibrate_static(W, p, s, signs, out)
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    q.calibrate_static(W, p, s, signs, out)
    torch.cuda.synchronize()
    assert torch.cuda.mem_get_info()[0] == free_before


def test_static_scratch_rejects_bad_arguments_without_launching():
    W, s, signs = _problem(8, 256, torch.float32, 3)
    sigma = torch.empty(128, dtype=torch.float32, device=DEV)
    p = q.make_params(W, 8, 256, 96, 256)  # block is not a power of two
    with pytest.raises(q.QamwError) as e:
        q.calibrate_static(W, p, s, signs, sigma)
    assert e.value.code == q.ERR_SHAPE
    torch.cuda.synchronize()
