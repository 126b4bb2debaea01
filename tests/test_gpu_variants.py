"""GPU side of the variants around the path: 16-bit metadata (Section 3.2), the decoder's optional
renormalisation (Section A.3), the alpha grid (Section B.2) and the on-disk blob."""
import os

import numpy as np
import pytest
import torch

from conftest import load_golden_codebook

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2605_26339_b200 import binding as q
    from paper_2605_26339_b200 import blob
    from paper_2605_26339_b200.model_codec import choose_alpha

DEV = "cuda:0"


def _bits(t):
    return t.cpu().view(torch.int16).numpy().view(np.uint16)


def _encode(W, act, alpha, block, K, round16=False):
    d_out, d_in = W.shape
    cbh = load_golden_codebook(K)
    cb = q.Codebook(cbh)
    s = torch.from_numpy(q.channel_scales(act, alpha)).to(DEV)
    signs = torch.from_numpy(q.make_signs(q.DEFAULT_SIGN_SEED, d_in)).to(DEV)
    Wd = W.to(DEV)
    p = q.make_params(Wd, d_out, d_in, block, K, 0, (q.packed_row_bytes(d_in, K) + 15) // 16 * 16)
    if round16:
        q.round_f16(s)
    sigma = torch.empty(d_in // 2, dtype=torch.float32, device=DEV)
    ws = torch.empty(q.calibrate_workspace_bytes(p), dtype=torch.uint8, device=DEV)
    q.calibrate(Wd, p, s, signs, sigma, ws)
    if round16:
        q.round_f16(sigma)
    packed = torch.empty((d_out, p.packed_row_stride), dtype=torch.uint8, device=DEV)
    norm = torch.empty(d_out, dtype=torch.float32, device=DEV)
    q.encode(Wd, p, s, signs, sigma, cb, packed, norm)
    if round16:
        q.round_f16(norm)
    return dict(cb=cb, cbh=cbh, s=s, signs=signs, W=Wd, p=p, sigma=sigma, packed=packed, norm=norm)


def _problem(seed, d_out=96, d_in=2048):
    g = torch.Generator().manual_seed(seed)
    W = (torch.randn((d_out, d_in), generator=g) * torch.exp(0.7 * torch.randn((d_out, 1), generator=g))).to(torch.bfloat16)
    act = torch.exp(torch.randn(d_in, generator=g)).numpy().astype(np.float32)
    return W, act


def test_round_f16_matches_oracle(orc):
    rng = np.random.default_rng(4)
    v = (rng.standard_normal(100003) * np.exp(rng.uniform(-22, 13, 100003))).astype(np.float32)
    v[:6] = [0.0, 65504.0, 65520.0, 2.0 ** -24, 2.0 ** -25, -1e9]
    t = torch.from_numpy(v.copy()).to(DEV)
    q.round_f16(t)
    assert np.array_equal(t.cpu().numpy(), orc.round_f16(v))


def test_renormalised_decode(orc):
    W, act = _problem(31)
    e = _encode(W, act, 0.3, 128, 256)
    adj = torch.empty_like(e["norm"])
    q.renorm_row_norms(e["packed"], e["norm"], e["sigma"], e["cb"], e["p"], adj)
    ref = orc.renorm_row_norms(e["packed"].cpu().numpy(), e["norm"].cpu().numpy(), e["sigma"].cpu().numpy(), e["cbh"], 2048)
    np.testing.assert_allclose(adj.cpu().numpy(), ref, rtol=2e-7)
    # decoding with the factors restores the stored norm of the scaled row
    what = torch.empty(W.shape, dtype=torch.bfloat16, device=DEV)
    q.decode(e["packed"], adj, e["s"], e["signs"], e["sigma"], e["cb"], e["p"], what)
    length = ((what.float() * e["s"]) ** 2).sum(1).sqrt()
    assert torch.allclose(length, e["norm"], rtol=2e-3)  # bf16 rounding of 2048 outputs
    q.decode(e["packed"], e["norm"], e["s"], e["signs"], e["sigma"], e["cb"], e["p"], what)
    plain = ((what.float() * e["s"]) ** 2).sum(1).sqrt()
    assert torch.allclose(plain, e["norm"] * e["norm"] / adj, rtol=2e-3)  # the plain decoder's length is r |yhat|
    assert not torch.allclose(plain, e["norm"], rtol=1e-4)


def test_f16_metadata_round_trip_through_a_blob(orc, tmp_path):
    """16-bit metadata end to end: scales and sigma rounded before encoding, norms after; the blob on
    disk (f16 metadata) decodes on the GPU to the very bits the in-memory arrays decode to, and the
    radial error added by the rounded norms stays within half an f16 ulp (2^-11 relative)."""
    W, act = _problem(32)
    e = _encode(W, act, 0.3, 128, 2048, round16=True)
    exact = _encode(W, act, 0.3, 128, 2048, round16=False)
    rel = (e["norm"] - exact["norm"]).abs() / exact["norm"]
    assert float(rel.max()) <= 2.0 ** -11 * 1.01 + 1e-3  # sigma / scales differ slightly too (<= 1e-3 on r)
    what = torch.empty(W.shape, dtype=torch.bfloat16, device=DEV)
    q.decode(e["packed"], e["norm"], e["s"], e["signs"], e["sigma"], e["cb"], e["p"], what)
    path = os.path.join(tmp_path, "m.qamw")
    size = blob.save_blob(path, d_out=96, d_in=2048, block=128, K=2048, alpha=0.3, sign_seed=q.DEFAULT_SIGN_SEED,
                          codebook=e["cbh"], sigma=e["sigma"].cpu().numpy(), row_norm=e["norm"].cpu().numpy(),
                          packed=e["packed"].cpu().numpy(), chan_scale=e["s"].cpu().numpy(), f16_metadata=True)
    b = blob.load_blob(path)
    cb2 = q.Codebook(b["codebook"])
    p2 = q.make_params(None, b["d_out"], b["d_in"], b["block"], b["K"], 0, b["packed_row_stride"])
    signs2 = torch.from_numpy(q.make_signs(b["sign_seed"], b["d_in"])).to(DEV)
    what2 = torch.empty(W.shape, dtype=torch.bfloat16, device=DEV)
    q.decode(torch.from_numpy(b["packed"]).to(DEV), torch.from_numpy(b["row_norm"]).to(DEV),
             torch.from_numpy(b["chan_scale"]).to(DEV), signs2, torch.from_numpy(b["sigma"]).to(DEV), cb2, p2, what2)
    assert np.array_equal(_bits(what), _bits(what2))
    # against the oracle on the same rounded metadata
    ref = orc.decode(b["packed"], b["row_norm"], 128, b["codebook"], b["chan_scale"], signs2.cpu().numpy(), b["sigma"], 2048)
    d = np.abs(_bits(what2).astype(np.int32) - ref.astype(np.int32))
    assert (d <= 1).mean() > 0.9998
    assert size < 96 * 2048 * 6 / 8 + 2048 * 8 + 8192  # about 5.5 bits per weight plus the codebook


def test_alpha_grid_picks_the_lowest_output_error(orc):
    W, act = _problem(33, 64, 1024)
    act[::50] *= 30.0  # a few loud channels make the scaling matter
    cb = q.Codebook(load_golden_codebook(256))
    best, scores = choose_alpha(W.to(DEV), torch.from_numpy(act).to(DEV), cb, 128)
    assert set(scores) == {0.0, 0.3, 0.5, 0.8} and best == min(scores, key=lambda a: scores[a][1])
    assert scores[best][1] < scores[0.0][1]  # scaling helps the activation-weighted error here
    # one grid point against the oracle's round trip
    s = orc.channel_scales(act, float(np.float32(0.5)))
    signs = orc.make_signs(q.DEFAULT_SIGN_SEED, 1024)
    Wb = _bits(W)
    sigma, _ = orc.calibrate(Wb, 128, s, signs)
    enc = orc.encode(Wb, 128, cb.host, s, signs, sigma)
    what = orc.decode(enc["packed"], enc["row_norm"], 128, cb.host, s, signs, sigma, 1024)
    d = orc.distortion(Wb, what, act)
    assert abs(np.sqrt(d[2] / d[3]) - scores[0.5][1]) < 2e-3 * scores[0.5][1]


@pytest.mark.parametrize("d_out,d_in,block,K,n_vec", [(300, 2048, 128, 2048, 1), (129, 5120, 128, 256, 4),
                                                      (64, 13824, 256, 2048, 2), (40, 1024, 32, 128, 1),
                                                      (33, 512, 1024 // 2, 4096, 1), (1000, 2048, 1024, 2048, 4),
                                                      (7, 64, 2, 64, 2), (50, 11008, 64, 1024, 1)])
def test_fused_decode_gemv(orc, d_out, d_in, block, K, n_vec):
    """y = W_hat x from the packed stream against the oracle's decoder (f64, before the bf16 rounding)
    followed by a plain matrix product.  The kernel accumulates in f32: the error of a row stays below
    1e-5 |w_hat_i| |x| (d_in terms, each product and sum rounded to 2^-24 relative)."""
    W, act = _problem(50 + n_vec, d_out, d_in)
    e = _encode(W, act, 0.3, block, K)
    g = torch.Generator().manual_seed(d_in)
    x = torch.randn((n_vec, d_in), generator=g)
    y = torch.full((d_out, n_vec), float("nan"), dtype=torch.float32, device=DEV)
    q.decode_gemv(e["packed"], e["norm"], e["s"], e["signs"], e["sigma"], e["cb"], e["p"], x.to(DEV), y)
    # the layout-agnostic kernel (taken for packed rows that are not 16-byte aligned) gives the same product
    y_general = torch.full_like(y, float("nan"))
    pg = q.make_params(None, d_out, d_in, block, K, q.FLAG_GENERAL_KERNELS, e["p"].packed_row_stride)
    q.decode_gemv(e["packed"], e["norm"], e["s"], e["signs"], e["sigma"], e["cb"], pg, x.to(DEV), y_general)
    _, w64 = orc.decode(e["packed"].cpu().numpy(), e["norm"].cpu().numpy(), block, e["cbh"], e["s"].cpu().numpy(),
                        e["signs"].cpu().numpy(), e["sigma"].cpu().numpy(), d_in, want_f64=True)
    ref = w64 @ x.numpy().astype(np.float64).T
    bound = 1e-5 * np.sqrt((w64 ** 2).sum(1))[:, None] * np.sqrt((x.numpy().astype(np.float64) ** 2).sum(1))[None, :]
    assert np.all(np.abs(y.cpu().numpy() - ref) <= bound + 1e-30)
    assert np.all(np.abs(y_general.cpu().numpy() - ref) <= bound + 1e-30)
    # and against the two-step pipeline of the paper (decode to bf16, then multiply): bf16 rounding only
    what = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=DEV)
    q.decode(e["packed"], e["norm"], e["s"], e["signs"], e["sigma"], e["cb"], e["p"], what)
    two_step = what.double() @ x.to(DEV).double().T
    assert torch.allclose(y.double(), two_step, rtol=0, atol=float(2.0 ** -7 * np.abs(ref).max() + 1e-30))


def test_fused_gemv_argument_errors():
    lv = load_golden_codebook(64)
    cb = q.Codebook(lv)
    dummy = torch.zeros(4096, dtype=torch.uint8, device=DEV)
    f = torch.zeros(4096, dtype=torch.float32, device=DEV)
    p = q.make_params(None, 4, 48, 16, 64)  # d_in not a multiple of 32
    with pytest.raises(q.QamwError) as e:
        q.decode_gemv(dummy, f, None, dummy, f, cb, p, f[:48].reshape(1, 48), f[:4].reshape(4, 1), dummy)
    assert e.value.code == q.ERR_SHAPE
    p = q.make_params(None, 4, 64, 16, 64)
    with pytest.raises(q.QamwError) as e:
        q.decode_gemv(dummy, f, None, dummy, f, cb, p, f[:192].reshape(3, 64), f[:12].reshape(4, 3), dummy)  # 3 vectors
    assert e.value.code == q.ERR_ARG


def test_step_replayed_as_a_cuda_graph_gives_the_same_bytes():
    """The batched step captured into one CUDA graph: replaying it reproduces the packed stream, the row
    norms, the decoded matrices and the distortion sums of the eager step bit for bit."""
    from paper_2605_26339_b200 import synth
    from paper_2605_26339_b200.model_codec import ModelCodec
    spec = synth.workload("cfg2", 256)
    mc = ModelCodec.from_synthetic(spec, torch.device(DEV), load_golden_codebook(256), layers=[0])
    mc.step()
    torch.cuda.synchronize()
    want = [(s.packed.clone(), s.row_norm.clone(), s.w_hat.clone(), s.dist.clone()) for s in mc.slots]
    graph = mc.capture_step()
    for s in mc.slots:
        s.packed.zero_(); s.row_norm.zero_(); s.w_hat.zero_(); s.dist.zero_()
    graph.replay()
    torch.cuda.synchronize()
    for s, (p, r, w, d) in zip(mc.slots, want):
        assert torch.equal(s.packed, p) and torch.equal(s.row_norm, r)
        assert torch.equal(s.w_hat.view(torch.int16), w.view(torch.int16)) and torch.equal(s.dist, d)
    assert int(mc.status.cpu()[0]) == 0
