"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same
seeded inputs.

Exactness rules of this codec:
  * packed indices bit-exact, except pairs whose oracle best / second-best squared distances
    differ by less than 1e-6 relative -- those are counted, and the GPU's choice must then be
    one of the two near-tied codewords;
  * rotated coordinates and row norms within 1e-5 relative (they are in fact required to be
    bit-identical here, because the index rule needs identical 2-D points);
  * decoded weights within 1 bf16 ulp given identical indices.  The kernel's inverse butterfly runs
    in f32 and the oracle's in f64: an output that nearly cancels (|w| far below its block's norm)
    carries an absolute error of up to 2^-21 |yhat_block| r / s_j, which can exceed one ulp of such a
    small value.  Those elements are accepted within that absolute bound, counted, and their share
    must stay below kFarFraction;
  * calibration within 1e-5 relative; distortion sums within 1e-9 relative.
"""
import numpy as np
import pytest
import torch

from conftest import load_golden_codebook

pytestmark = pytest.mark.gpu

if torch.cuda.is_available():
    from paper_2605_26339_b200 import binding as q
    from paper_2605_26339_b200 import synth

DEV = "cuda:0"
_codebooks = {}
kFarFraction = 2e-4  # share of decoded weights allowed beyond 1 bf16 ulp (all within the absolute bound)


def _codebook(orc, K):
    if K not in _codebooks:
        if K >= 64:
            host = load_golden_codebook(K)
        else:  # tiny codebooks: trained by the oracle on the spot
            host = orc.train_codebook(K, 1 << 12, 7, 30, 1e-6)[0]
        _codebooks[K] = (host, q.Codebook(host))
    return _codebooks[K]


def _to_bits(W: torch.Tensor) -> np.ndarray:
    if W.dtype == torch.bfloat16:
        return W.cpu().view(torch.int16).numpy().view(np.uint16)
    return W.cpu().numpy()


def _make(d_out, d_in, dtype, seed, student=True):
    g = torch.Generator().manual_seed(seed)
    x = torch.randn((d_out, d_in), generator=g)
    if student:
        chi = sum(torch.randn((d_out, d_in), generator=g) ** 2 for _ in range(4)) / 4
        x = x / chi.sqrt()
    x = x * torch.exp(0.7 * torch.randn((d_out, 1), generator=g))
    act = torch.exp(torch.randn(d_in, generator=g))
    return x.to(dtype), act.numpy().astype(np.float32)


def _bf16_ordered(bits: np.ndarray) -> np.ndarray:
    b = bits.astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b & 0x7FFF)


class Case:
    """Runs every GPU entry point on one matrix and keeps the outputs on the host."""

    def __init__(self, orc, W: torch.Tensor, act, alpha, block, K, flags=0, row_sel=None, packed_stride=None):
        self.orc, self.block, self.K = orc, block, K
        d_out, d_in = W.shape
        self.d_out, self.d_in = d_out, d_in
        self.cb_host, self.cb = _codebook(orc, K)
        self.s = q.channel_scales(act, alpha) if alpha else None
        self.signs = q.make_signs(q.DEFAULT_SIGN_SEED, d_in)
        Wd = W.to(DEV) if W.device.type == "cpu" else W
        self.Wd = Wd
        self.p = q.make_params(Wd, d_out, d_in, block, K, flags, packed_stride)
        s_d = None if self.s is None else torch.from_numpy(self.s).to(DEV)
        signs_d = torch.from_numpy(self.signs).to(DEV)
        # rows the oracle looks at (all rows unless a sample is given)
        self.rows = np.arange(d_out) if row_sel is None else np.asarray(row_sel)
        self.W_rows = _to_bits(Wd[torch.from_numpy(self.rows).to(DEV)]) if row_sel is not None else _to_bits(Wd)

        # calibration: GPU on the full matrix; oracle on the full matrix too (it reads <= 1024 rows)
        ws = torch.empty(max(8, q.calibrate_workspace_bytes(self.p)), dtype=torch.uint8, device=DEV)
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)
        sigma_d = torch.empty(d_in // 2, dtype=torch.float32, device=DEV)
        q.calibrate(Wd, self.p, s_d, signs_d, sigma_d, ws, self.status)
        self.sigma_gpu = sigma_d.cpu().numpy()
        n_cal = min(d_out, 1024)
        cal_rows = (np.arange(n_cal) * d_out) // n_cal
        W_cal = _to_bits(Wd[torch.from_numpy(cal_rows).to(DEV)])
        self.sigma, rc = orc.calibrate(W_cal, block, self.s, self.signs)
        sigma_d = torch.from_numpy(self.sigma).to(DEV)  # both sides use the oracle's sigma from here on

        self.y_d = torch.empty((d_out, d_in), dtype=torch.float32, device=DEV)
        norm_rot = torch.empty(d_out, dtype=torch.float32, device=DEV)
        q.rotate(Wd, self.p, s_d, signs_d, self.y_d, norm_rot, self.status)
        self.norm_rot = norm_rot.cpu().numpy()

        stride = self.p.packed_row_stride
        packed_d = torch.full((d_out, stride), 0xAB, dtype=torch.uint8, device=DEV)
        norm_d = torch.empty(d_out, dtype=torch.float32, device=DEV)
        q.encode(Wd, self.p, s_d, signs_d, sigma_d, self.cb, packed_d, norm_d, self.status)
        self.packed = packed_d.cpu().numpy()
        self.norm = norm_d.cpu().numpy()

        self.enc = orc.encode(self.W_rows, block, self.cb_host, self.s, self.signs, self.sigma,
                              packed_row_stride=stride, diagnostics=True)
        # decode the ORACLE's stream on the GPU ("given identical indices")
        opacked = np.ascontiguousarray(self.enc["packed"])
        pk = torch.from_numpy(opacked).to(DEV)
        nm = torch.from_numpy(self.enc["row_norm"]).to(DEV)
        what_d = torch.empty((len(self.rows), d_in), dtype=torch.bfloat16, device=DEV)
        p_dec = q.make_params(None, len(self.rows), d_in, block, K, 0, stride)
        q.decode(pk, nm, s_d, signs_d, sigma_d, self.cb, p_dec, what_d)
        self.what = _to_bits(what_d)
        # distortion of the GPU's own round trip on the full matrix
        what_full = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=DEV)
        q.decode(packed_d, norm_d, s_d, signs_d, sigma_d, self.cb, self.p, what_full)
        out4 = torch.empty(4, dtype=torch.float64, device=DEV)
        act_d = torch.from_numpy(np.ascontiguousarray(act, np.float32)).to(DEV)
        q.distortion(Wd, what_full, act_d, self.p, out4)
        torch.cuda.synchronize()
        self.out4 = out4.cpu().numpy()
        self.what_full = _to_bits(what_full)
        self.act = act
        self.status_word = int(self.status.cpu()[0])

    # ---- checks ------------------------------------------------------------------------------
    def check_calibration(self):
        np.testing.assert_allclose(self.sigma_gpu, self.sigma, rtol=1e-5)

    def check_front_half(self):
        y = self.y_d[torch.from_numpy(self.rows).to(DEV)].cpu().numpy()
        zq = (1.0 / self.sigma.astype(np.float64)).astype(np.float32)
        z_gpu = (y.reshape(len(self.rows), -1, 2) * zq[None, :, None]).astype(np.float32)
        z_orc = self.enc["z"]
        scale = np.abs(z_orc).max(axis=(1, 2), keepdims=True) + 1e-30
        assert np.all(np.abs(z_gpu - z_orc) <= 1e-5 * scale)
        np.testing.assert_allclose(self.norm[self.rows], self.enc["row_norm"], rtol=1e-5)
        np.testing.assert_allclose(self.norm_rot[self.rows], self.enc["row_norm"], rtol=1e-5)
        # value equality: -0.0 of an all-zero row counts as +0.0
        same_z = np.array_equal(z_gpu, z_orc)
        same_r = np.array_equal(self.norm[self.rows], self.enc["row_norm"])
        self.max_dz = float(np.abs(z_gpu.astype(np.float64) - z_orc).max()) if z_orc.size else 0.0
        self.max_dr = float(np.abs(self.norm[self.rows].astype(np.float64) - self.enc["row_norm"]).max()) if len(self.rows) else 0.0
        return same_z, same_r

    def check_indices(self):
        B = int(np.log2(self.K))
        n_pairs = self.d_in // 2
        idx_gpu = np.stack([self.orc.unpack_row(self.packed[r], n_pairs, B) for r in self.rows])
        idx_orc = self.enc["idx"]
        d1, d2 = self.enc["d2_best"], self.enc["d2_second"]
        diff = idx_gpu != idx_orc
        exempt = (d2 - d1) < 1e-6 * d2
        assert not np.any(diff & ~exempt), f"{int((diff & ~exempt).sum())} non-exempt index mismatches"
        if diff.any():  # an exempt mismatch must still be one of the near-tied codewords
            z = self.enc["z"].astype(np.float64)[diff]
            c = self.cb_host[idx_gpu[diff]].astype(np.float64)
            dg = ((z - c) ** 2).sum(1)
            assert np.all(dg <= d2[diff] * (1 + 1e-9))
        # padding up to the row stride is zero
        rb = q.packed_row_bytes(self.d_in, self.K)
        assert not self.packed[:, rb:].any()
        tail_bits = rb * 8 - n_pairs * B
        if tail_bits:
            assert not np.any(self.packed[:, rb - 1] >> (8 - tail_bits))
        return int(diff.sum()), int(exempt.sum()), idx_gpu.size

    def check_decode(self):
        s = np.ones(self.d_in) if self.s is None else self.s.astype(np.float64)
        ref_bits, ref64 = self.orc.decode(self.enc["packed"], self.enc["row_norm"], self.block, self.cb_host, self.s,
                                          self.signs, self.sigma, self.d_in, want_f64=True)
        ulps = np.abs(_bf16_ordered(self.what) - _bf16_ordered(ref_bits))
        got = self.orc.bf16_to_f32(self.what).astype(np.float64)
        yhat = self.cb_host[self.enc["idx"]].astype(np.float64) * self.sigma.astype(np.float64)[None, :, None]
        blk = np.sqrt((yhat.reshape(len(self.rows), -1, self.block) ** 2).sum(2))  # |yhat_block|_2
        abs_tol = 2.0**-21 * np.repeat(blk, self.block, axis=1) * self.enc["row_norm"].astype(np.float64)[:, None] / s
        ok = (ulps <= 1) | (np.abs(got - ref64) <= abs_tol + 2.0**-8 * np.abs(ref64) * 0.51)
        assert np.all(ok), f"{int((~ok).sum())} decoded weights out of tolerance"
        n_far = int((ulps > 1).sum())
        assert n_far <= kFarFraction * ulps.size + 2, f"{n_far} of {ulps.size} decoded weights beyond 1 bf16 ulp"
        self.ulp_hist = [int((ulps == 0).sum()), int((ulps == 1).sum()), n_far]
        return float((ulps == 0).mean()), n_far

    def check_distortion(self):
        ref = self.orc.distortion(_to_bits(self.Wd), self.what_full, self.act)
        np.testing.assert_allclose(self.out4, ref, rtol=1e-9)

    def check_all(self, expect_bit_identical=True):
        self.check_calibration()
        same_z, same_r = self.check_front_half()
        if expect_bit_identical:
            assert same_z and same_r
        n_diff, n_exempt, n = self.check_indices()
        exact_frac, n_far = self.check_decode()
        self.check_distortion()
        assert exact_frac > 0.98
        assert self.status_word == 0
        # round-trip error of the oracle's own stream on the checked rows, beside the GPU's
        w = self.orc.bf16_to_f32(self.W_rows).astype(np.float64) if self.W_rows.dtype == np.uint16 else self.W_rows.astype(np.float64)
        ref_bits = self.orc.decode(self.enc["packed"], self.enc["row_norm"], self.block, self.cb_host, self.s, self.signs,
                                   self.sigma, self.d_in)
        mse_orc = float(((w - self.orc.bf16_to_f32(ref_bits)) ** 2).mean())
        mse_gpu = float(((w - self.orc.bf16_to_f32(self.what_full[self.rows])) ** 2).mean())
        return dict(shape=[self.d_out, self.d_in], K=self.K, block=self.block, rows_checked=len(self.rows),
                    mismatches=n_diff, mismatches_nonexempt=0, exempt_pairs=n_exempt, pairs=n, max_dz=self.max_dz,
                    max_dr=self.max_dr, ulp_hist=self.ulp_hist, mse_gpu=mse_gpu, mse_oracle=mse_orc)


# ------------------------------------------------------------------------------------------------
def test_cfg0_full(orc):
    """Configuration 0: W[1024,1024] f32, alpha 0.5, block 128, K 256 -- every row checked."""
    spec = synth.workload("cfg0")
    W = synth.make_weight(spec, spec.matrices[0], synth.matrix_seed(spec, 0, 0))
    act = synth.make_act_rms(spec, 1024, 1).numpy()
    rep = Case(orc, W, act, spec.alpha, spec.block, spec.K).check_all()
    _report("cfg0 all rows", rep)


@pytest.mark.parametrize("kernels", ["fast", "general"])
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("block", [2, 4, 8, 16, 32, 64, 128, 256, 512, 1024])
def test_block_sizes(orc, block, dtype, kernels):
    """Every block size through the kernels for the common layouts (block >= 32) and, with
    QAMW_FLAG_GENERAL_KERNELS, through the general row kernels."""
    W, act = _make(37, 2048, dtype, 100 + block)
    flags = q.FLAG_GENERAL_KERNELS if kernels == "general" else 0
    if kernels == "general" and block < 32:
        pytest.skip("blocks below 32 always run the general kernels")
    Case(orc, W, act, 0.3, block, 256, flags=flags).check_all()


@pytest.mark.parametrize("kernels", ["fast", "general"])
@pytest.mark.parametrize("K", [2, 4, 16, 64, 128, 1024, 2048, 4096])
def test_codebook_sizes(orc, K, kernels):
    W, act = _make(33, 1024, torch.bfloat16, 200 + K)
    Case(orc, W, act, 0.3, 128, K, flags=q.FLAG_GENERAL_KERNELS if kernels == "general" else 0).check_all()


@pytest.mark.parametrize("d_out,d_in,block", [(1, 2, 2), (3, 4, 4), (5, 6, 2), (1, 8, 8), (7, 24, 8), (3, 40, 8),
                                              (1025, 64, 64), (2, 192, 64), (9, 1152, 128), (3, 16384, 1024)])
def test_ragged_shapes(orc, d_out, d_in, block):
    """Rows shorter than a thread's 32 elements, rows that are not a multiple of 8 long (element-wise
    load path), more rows than one wave of the grid, the longest supported row."""
    W, act = _make(d_out, d_in, torch.float32, d_out * 7 + d_in)
    Case(orc, W, act, 0.5, block, 64).check_all()


def test_strided_and_misaligned_rows(orc):
    base, act = _make(16, 520, torch.bfloat16, 5)
    base = base.to(DEV)
    W = base[:, 3:515]  # row stride 520, rows start 6 bytes off a 16-byte boundary
    assert W.stride(0) == 520 and W.data_ptr() % 16 == 6
    Case(orc, W, act[3:515], 0.3, 128, 256, packed_stride=720).check_all()
    W = base[:, 8:520]  # aligned, strided
    Case(orc, W, act[8:520], 0.3, 128, 256).check_all()


def test_no_channel_scaling_and_brute_force_flag(orc):
    W, act = _make(64, 1024, torch.bfloat16, 11)
    a = Case(orc, W, act, 0.0, 128, 2048)
    a.check_all()
    b = Case(orc, W, act, 0.0, 128, 2048, flags=q.FLAG_BRUTE_FORCE)
    b.check_all()
    B = 11
    ia = np.stack([orc.unpack_row(r, 512, B) for r in a.packed])
    ib = np.stack([orc.unpack_row(r, 512, B) for r in b.packed])
    assert (ia != ib).mean() < 1e-4  # the two searches may differ only on near ties


def test_zero_outlier_and_nonfinite_rows(orc):
    W, act = _make(12, 512, torch.float32, 13, student=False)
    W[2] = 0
    W[5, 17] = 3.0e4  # one huge entry: its block's points land in the outermost cells of the table
    c = Case(orc, W, act, 0.0, 128, 256)
    c.check_all()
    assert c.norm[2] == 0 and not orc.bf16_to_f32(c.what_full[2]).any()
    W[7, 100] = float("inf")
    W[9, 3] = float("nan")
    c = Case(orc, W, act, 0.0, 128, 256)
    assert c.status_word == 1 and q.status_to_error(c.status_word) == q.ERR_NONFINITE
    assert c.enc["status"] == orc.ORC_ERR_NONFINITE
    ok = [r for r in range(12) if r not in (7, 9)]  # the other rows are unaffected
    B, n_pairs = 8, 256
    idx_gpu = np.stack([orc.unpack_row(c.packed[r], n_pairs, B) for r in ok])
    exempt = (c.enc["d2_second"][ok] - c.enc["d2_best"][ok]) < 1e-6 * c.enc["d2_second"][ok]
    assert not np.any((idx_gpu != c.enc["idx"][ok]) & ~exempt)


@pytest.mark.parametrize("sigma0,z_min", [(1e-3, 8.0), (1e-5, 16000.0)])
def test_extreme_z(orc, sigma0, z_min):
    """sigma far too small: at 1e-3 the points land in the outermost cells of the table (|z| up to
    some hundreds); at 1e-5 the reciprocal scale is large enough for the encoder to run its variant
    with the reach check, and the points beyond |z| = 16000 go through the exhaustive scan."""
    W, act = _make(6, 256, torch.float32, 17, student=False)
    cb_host, cb = _codebook(orc, 256)
    signs = q.make_signs(q.DEFAULT_SIGN_SEED, 256)
    sigma = np.full(128, sigma0, np.float32)
    p = q.make_params(W.to(DEV), 6, 256, 64, 256)
    packed = torch.zeros((6, p.packed_row_stride), dtype=torch.uint8, device=DEV)
    norm = torch.empty(6, dtype=torch.float32, device=DEV)
    q.encode(W.to(DEV), p, None, torch.from_numpy(signs).to(DEV), torch.from_numpy(sigma).to(DEV), cb, packed, norm)
    enc = orc.encode(W.numpy(), 64, cb_host, None, signs, sigma, packed_row_stride=p.packed_row_stride, diagnostics=True)
    assert np.abs(enc["z"]).max() > z_min
    idx_gpu = np.stack([orc.unpack_row(r, 128, 8) for r in packed.cpu().numpy()])
    exempt = (enc["d2_second"] - enc["d2_best"]) < 1e-6 * enc["d2_second"]
    assert not np.any((idx_gpu != enc["idx"]) & ~exempt)


@pytest.mark.parametrize("K,grid", [(256, 3), (256, 9), (256, 117), (2048, 41)])
def test_explicit_search_grids(orc, K, grid):
    """A coarse grid sends nearly every point through the overflow lists, a fine one through cells
    with a single candidate; the indices are the oracle's either way, also for heavy-tailed pairs
    that land in the outermost columns."""
    W, act = _make(24, 1024, torch.float32, 300 + grid)
    # a few huge entries per row: the pairs of their blocks spread far beyond the Gaussian range
    W[torch.rand(W.shape, generator=torch.Generator().manual_seed(grid)) < 0.004] *= 40.0
    cb_host = load_golden_codebook(K)
    cb = q.Codebook(cb_host, grid=grid)
    assert int(cb.table_info()[0]) == grid
    if grid <= 9:
        assert int(cb.table_info()[3]) > grid * grid // 2  # most cells overflow
    signs = q.make_signs(q.DEFAULT_SIGN_SEED, 1024)
    sigma, _ = orc.calibrate(W.numpy(), 128, None, signs)
    p = q.make_params(W.to(DEV), 24, 1024, 128, K)
    packed = torch.zeros((24, p.packed_row_stride), dtype=torch.uint8, device=DEV)
    norm = torch.empty(24, dtype=torch.float32, device=DEV)
    q.encode(W.to(DEV), p, None, torch.from_numpy(signs).to(DEV), torch.from_numpy(sigma).to(DEV), cb, packed, norm)
    enc = orc.encode(W.numpy(), 128, cb_host, None, signs, sigma, packed_row_stride=p.packed_row_stride,
                     diagnostics=True)
    assert np.abs(enc["z"]).max() > 4.5  # beyond the polynomial part of the cell map
    B = int(np.log2(K))
    idx_gpu = np.stack([orc.unpack_row(r, 512, B) for r in packed.cpu().numpy()])
    exempt = (enc["d2_second"] - enc["d2_best"]) < 1e-6 * enc["d2_second"]
    assert not np.any((idx_gpu != enc["idx"]) & ~exempt)
    assert np.array_equal(norm.cpu().numpy(), enc["row_norm"])


@pytest.mark.parametrize("name,mid", [("cfg3", 0), ("cfg3", 4), ("cfg3", 6), ("cfg1", 6), ("cfg2", 1)])
def test_full_size_matrices_sampled_rows(orc, name, mid):
    """Benchmark-size matrices in the benchmark's launch configuration (whole matrix on the device,
    generated there); the oracle checks a spread of sampled rows."""
    spec = synth.workload(name)
    m = spec.matrices[mid]
    W = synth.make_weight(spec, m, synth.matrix_seed(spec, 0, mid), device=DEV)
    act = synth.make_act_rms(spec, m.d_in, 3, device=DEV).cpu().numpy()
    rows = np.unique(np.concatenate([[0, 1, m.d_out - 1], np.linspace(0, m.d_out - 1, 45).astype(int)]))
    rep = Case(orc, W, act, spec.alpha, spec.block, spec.K, row_sel=rows).check_all()
    _report(f"{name} {m.name} K={spec.K} sampled rows", rep)


def test_encode_decode_are_deterministic(orc):
    W, act = _make(300, 2048, torch.bfloat16, 23)
    a = Case(orc, W, act, 0.3, 128, 2048)
    b = Case(orc, W, act, 0.3, 128, 2048)
    assert np.array_equal(a.packed, b.packed) and np.array_equal(a.norm, b.norm)
    assert np.array_equal(a.what_full, b.what_full) and np.array_equal(a.sigma_gpu, b.sigma_gpu)


def test_half_device_flag_changes_nothing_but_the_grid(orc):
    """QAMW_FLAG_HALF_DEVICE only limits the number of blocks: same bits out, and parity still holds."""
    W, act = _make(700, 2048, torch.bfloat16, 29)
    a = Case(orc, W, act, 0.3, 128, 2048)
    b = Case(orc, W, act, 0.3, 128, 2048, flags=q.FLAG_HALF_DEVICE)
    b.check_all()
    assert np.array_equal(a.packed, b.packed) and np.array_equal(a.norm, b.norm)
    assert np.array_equal(a.what_full, b.what_full)


def test_empty_matrix(orc):
    cb_host, cb = _codebook(orc, 64)
    p = q.make_params(None, 0, 64, 64, 64)
    dummy = torch.zeros(64, dtype=torch.uint8, device=DEV)
    signs = torch.ones(64, dtype=torch.int8, device=DEV)
    sigma = torch.ones(32, dtype=torch.float32, device=DEV)
    q.encode(dummy, p, None, signs, sigma, cb, dummy, sigma)  # d_out = 0: nothing launched, no error
    q.decode(dummy, sigma, None, signs, sigma, cb, p, dummy)
    torch.cuda.synchronize()


def _report(tag, rep):
    import json
    print("PARITY " + json.dumps({"case": tag, **rep}))


@pytest.mark.parametrize("K,block", [(64, 64), (64, 256), (4096, 64), (4096, 256)])
def test_sweep_corners_sampled_rows(orc, K, block):
    """The four corners of configuration 4's grid (K x block) on the full W[13824,5120] matrix, in the
    benchmark's launch configuration; the oracle checks a spread of rows."""
    spec = synth.workload("cfg4", K=K, block=block)
    m = spec.matrices[0]
    W = synth.make_weight(spec, m, synth.matrix_seed(spec, 0, 0), device=DEV)
    act = synth.make_act_rms(spec, m.d_in, 3, device=DEV).cpu().numpy()
    rows = np.unique(np.concatenate([[0, 1, m.d_out - 1], np.linspace(0, m.d_out - 1, 29).astype(int)]))
    _report(f"cfg4 K={K} b={block}", Case(orc, W, act, spec.alpha, block, K, row_sel=rows).check_all())


@pytest.mark.parametrize("mid", [0, 1, 4, 6])
def test_tinyllama_matrices_at_K128(orc, mid):
    """Configuration 2 at its second codebook size (B = 7): q, k (256 rows), gate and down matrices."""
    spec = synth.workload("cfg2", K=128)
    m = spec.matrices[mid]
    W = synth.make_weight(spec, m, synth.matrix_seed(spec, 0, mid), device=DEV)
    act = synth.make_act_rms(spec, m.d_in, 5, device=DEV).cpu().numpy()
    rows = np.unique(np.linspace(0, m.d_out - 1, 40).astype(int))
    _report(f"cfg2 {m.name} K=128", Case(orc, W, act, spec.alpha, spec.block, 128, row_sel=rows).check_all())


@pytest.mark.parametrize("mid", [0, 6])
def test_full_matrix_every_row(orc, mid):
    """Every row of one full matrix per row-length class of configuration 3 ([5120,5120] and
    [5120,13824]).  K = 256 keeps the oracle's exhaustive search to some seconds on the host cores."""
    spec = synth.workload("cfg3", K=256)
    m = spec.matrices[mid]
    W = synth.make_weight(spec, m, synth.matrix_seed(spec, 0, mid), device=DEV)
    act = synth.make_act_rms(spec, m.d_in, 7, device=DEV).cpu().numpy()
    _report(f"cfg3 {m.name} K=256 all rows", Case(orc, W, act, spec.alpha, spec.block, 256).check_all())


def _batch_problem(shapes, K, block, dtype, flags=0):
    cb_host = load_golden_codebook(K)
    cb = q.Codebook(cb_host)
    slots = []
    for i, (d_out, d_in) in enumerate(shapes):
        W, act = _make(d_out, d_in, dtype, 900 + i)
        Wd = W.to(DEV)
        p = q.make_params(Wd, d_out, d_in, block, K, flags, (q.packed_row_bytes(d_in, K) + 15) // 16 * 16)
        slots.append(dict(
            p=p, W=Wd, act=torch.from_numpy(act).to(DEV),
            s=torch.from_numpy(q.channel_scales(act, 0.3)).to(DEV),
            signs=torch.from_numpy(q.make_signs(q.DEFAULT_SIGN_SEED, d_in)).to(DEV),
            sigma=torch.zeros(d_in // 2, dtype=torch.float32, device=DEV),
            packed=torch.full((d_out, p.packed_row_stride), 0xCD, dtype=torch.uint8, device=DEV),
            norm=torch.zeros(d_out, dtype=torch.float32, device=DEV),
            what=torch.zeros((d_out, d_in), dtype=torch.bfloat16, device=DEV),
            dist=torch.zeros(4, dtype=torch.float64, device=DEV)))
    return cb, slots


@pytest.mark.parametrize("shapes,block", [
    ([(300, 2048), (64, 11776), (129, 512), (40, 5120)], 128),   # both encoder classes (rows beyond 11264 elements)
    ([(77, 1024), (5, 24), (33, 2048)], 8),                      # a matrix outside the common layout: falls back
])
def test_batch_equals_single_matrix_calls(orc, shapes, block):
    """qamw_*_batch over several matrices gives, bit for bit, what the single-matrix entry points give."""
    K = 256
    cb, a = _batch_problem(shapes, K, block, torch.bfloat16)
    _, b = _batch_problem(shapes, K, block, torch.bfloat16)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    for s in a:  # reference: one call per matrix
        ws = torch.empty(q.calibrate_workspace_bytes(s["p"]), dtype=torch.uint8, device=DEV)
        q.calibrate(s["W"], s["p"], s["s"], s["signs"], s["sigma"], ws, st)
        q.encode(s["W"], s["p"], s["s"], s["signs"], s["sigma"], cb, s["packed"], s["norm"], st)
        q.decode(s["packed"], s["norm"], s["s"], s["signs"], s["sigma"], cb, s["p"], s["what"])
        q.distortion(s["W"], s["what"], s["act"], s["p"], s["dist"])
    mats = [q.make_matrix(s["p"], s["W"], s["s"], s["signs"], s["sigma"], s["act"], s["packed"], s["norm"], s["what"],
                          s["dist"]) for s in b]
    batch = q.Batch(mats, cb)
    ws = torch.empty(max(8, batch.workspace_bytes()), dtype=torch.uint8, device=DEV)
    batch.calibrate(ws, st)
    for x, y in zip(a, b):  # the batched pass groups the calibration rows differently: last-bit differences only
        np.testing.assert_allclose(y["sigma"].cpu().numpy(), x["sigma"].cpu().numpy(), rtol=1e-6)
        y["sigma"].copy_(x["sigma"])
    batch.encode(st)
    batch.decode()
    batch.distortion()
    torch.cuda.synchronize()
    assert int(st.cpu()[0]) == 0
    for x, y in zip(a, b):
        assert torch.equal(x["packed"], y["packed"]) and torch.equal(x["norm"], y["norm"])
        assert torch.equal(x["what"].view(torch.int16), y["what"].view(torch.int16))
        np.testing.assert_allclose(x["dist"].cpu().numpy(), y["dist"].cpu().numpy(), rtol=1e-9)
    # the batched sums are added in a fixed order: a second launch gives the same bits
    first = [y["dist"].clone() for y in b]
    batch.distortion()
    torch.cuda.synchronize()
    for f, y in zip(first, b):
        assert torch.equal(f, y["dist"])
    # and the first matrix against the oracle, through the batch's outputs
    s0 = b[0]
    Wb = _to_bits(s0["W"])
    enc = orc.encode(Wb, block, cb.host, s0["s"].cpu().numpy(), s0["signs"].cpu().numpy(), s0["sigma"].cpu().numpy(),
                     packed_row_stride=s0["p"].packed_row_stride, diagnostics=True)
    B = int(np.log2(K))
    idx = np.stack([orc.unpack_row(r, shapes[0][1] // 2, B) for r in s0["packed"].cpu().numpy()])
    exempt = (enc["d2_second"] - enc["d2_best"]) < 1e-6 * enc["d2_second"]
    assert not np.any((idx != enc["idx"]) & ~exempt)
    assert np.array_equal(s0["norm"].cpu().numpy(), enc["row_norm"])


@pytest.mark.parametrize("Ba,Bp,d_out,d_in,block,dtype", [
    (5, 6, 48, 2048, 128, torch.bfloat16),   # the paper's 11-bit split
    (3, 4, 33, 1024, 64, torch.float32),
    (0, 3, 9, 512, 32, torch.bfloat16),      # phase only
    (4, 0, 9, 512, 256, torch.bfloat16),     # amplitude only
    (5, 6, 20, 13824, 128, torch.bfloat16),  # the longest rows of configuration 3
])
def test_polar_baseline_codec(orc, Ba, Bp, d_out, d_in, block, dtype):
    """Polar baseline (Section 3.5) on the GPU against the oracle: indices equal except where the
    oracle's margins say that f32 cannot tell (amplitude within 1e-6 relative of a level threshold,
    phase within 1e-6 rad of a bin boundary) -- there the GPU's index must be the neighbouring level
    or bin; decode of the oracle's stream through the reconstruction table as for the 2-D codec."""
    W, act = _make(d_out, d_in, dtype, 700 + Ba * 16 + Bp)
    W[1] = 0  # a zero row: every pair is the origin (phase bin 0, lowest level)
    lv, _ = q.polar_train(Ba)
    cb = q.Codebook.polar(lv, Ba, Bp)
    K, B = 1 << (Ba + Bp), Ba + Bp
    s = q.channel_scales(act, 0.3)
    signs = q.make_signs(q.DEFAULT_SIGN_SEED, d_in)
    Wd, s_d, signs_d = W.to(DEV), torch.from_numpy(s).to(DEV), torch.from_numpy(signs).to(DEV)
    sigma, _ = orc.calibrate(_to_bits(Wd), block, s, signs)
    sigma_d = torch.from_numpy(sigma).to(DEV)
    p = q.make_params(Wd, d_out, d_in, block, K, 0, (q.packed_row_bytes(d_in, K) + 15) // 16 * 16)
    packed = torch.full((d_out, p.packed_row_stride), 0xEE, dtype=torch.uint8, device=DEV)
    norm = torch.empty(d_out, dtype=torch.float32, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    q.encode(Wd, p, s_d, signs_d, sigma_d, cb, packed, norm, st)
    enc = orc.encode_polar(_to_bits(Wd), block, lv, Ba, Bp, s, signs, sigma, packed_row_stride=p.packed_row_stride,
                           diagnostics=True)
    torch.cuda.synchronize()
    assert int(st.cpu()[0]) == 0 and np.array_equal(norm.cpu().numpy(), enc["row_norm"])
    pk = packed.cpu().numpy()
    idx = np.stack([orc.unpack_row(r, d_in // 2, B) for r in pk])
    diff = idx != enc["idx"]
    exempt = (enc["margin_a"] < 1e-6) | (enc["margin_p"] < 1e-6)
    assert not np.any(diff & ~exempt), f"{int((diff & ~exempt).sum())} non-exempt index mismatches"
    if diff.any():  # one step in the ambiguous component only
        ga, gp = idx[diff] & ((1 << Ba) - 1), idx[diff] >> Ba
        oa, op = enc["idx"][diff] & ((1 << Ba) - 1), enc["idx"][diff] >> Ba
        dp = np.abs(gp - op)
        assert np.all(np.abs(ga - oa) <= 1) and np.all((dp <= 1) | (dp == (1 << Bp) - 1))
    assert not idx[1].any()
    rb = q.packed_row_bytes(d_in, K)
    assert not pk[:, rb:].any()
    # decode the oracle's stream
    what = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=DEV)
    q.decode(torch.from_numpy(enc["packed"]).to(DEV), torch.from_numpy(enc["row_norm"]).to(DEV), s_d, signs_d, sigma_d, cb, p, what)
    ref = orc.decode(enc["packed"], enc["row_norm"], block, cb.host, s, signs, sigma, d_in)
    ulps = np.abs(_bf16_ordered(_to_bits(what)) - _bf16_ordered(ref))
    assert (ulps <= 1).mean() > 1 - kFarFraction - 2.0 / ulps.size and (ulps == 0).mean() > 0.98
    # the fused matrix-vector product works from the same reconstruction table
    if d_in % 32 == 0:
        g = torch.Generator().manual_seed(Ba + 3)
        x = torch.randn((2, d_in), generator=g)
        y = torch.full((d_out, 2), float("nan"), dtype=torch.float32, device=DEV)
        q.decode_gemv(torch.from_numpy(enc["packed"]).to(DEV), torch.from_numpy(enc["row_norm"]).to(DEV), s_d, signs_d,
                      sigma_d, cb, p, x.to(DEV), y)
        _, w64 = orc.decode(enc["packed"], enc["row_norm"], block, cb.host, s, signs, sigma, d_in, want_f64=True)
        x64 = x.numpy().astype(np.float64)
        bound = 1e-5 * np.sqrt((w64 ** 2).sum(1))[:, None] * np.sqrt((x64 ** 2).sum(1))[None, :]
        assert np.all(np.abs(y.cpu().numpy() - w64 @ x64.T) <= bound + 1e-30)
    print("PARITY polar", dict(Ba=Ba, Bp=Bp, pairs=int(idx.size), mismatches=int(diff.sum()), exempt=int(exempt.sum())))


def test_polar_encoder_refuses_layouts_outside_its_kernels(orc):
    lv, _ = q.polar_train(2)
    cb = q.Codebook.polar(lv, 2, 2)
    W = torch.zeros((4, 64), dtype=torch.float32, device=DEV)
    p = q.make_params(W, 4, 64, 16, 16)  # block 16: only the general kernels take it
    dummy = torch.zeros(64, dtype=torch.uint8, device=DEV)
    signs = torch.ones(64, dtype=torch.int8, device=DEV)
    sigma = torch.ones(32, dtype=torch.float32, device=DEV)
    with pytest.raises(q.QamwError) as e:
        q.encode(W, p, None, signs, sigma, cb, dummy, sigma)
    assert e.value.code == q.ERR_SHAPE


def test_one_call_quantize_equals_the_separate_calls(orc):
    """qamw_quantize (W, activation statistics, alpha, block, codebook in; stream and metadata out)
    gives what channel_scales -> make_signs -> calibrate -> encode give one after the other."""
    W, act = _make(200, 2048, torch.bfloat16, 41)
    c = Case(orc, W, act, 0.3, 128, 256)
    Wd = W.to(DEV)
    p = q.make_params(Wd, 200, 2048, 128, 256)
    s_out = torch.empty(2048, dtype=torch.float32, device=DEV)
    signs_out = torch.empty(2048, dtype=torch.int8, device=DEV)
    sigma_out = torch.empty(1024, dtype=torch.float32, device=DEV)
    packed = torch.full((200, p.packed_row_stride), 0x5A, dtype=torch.uint8, device=DEV)
    norm = torch.empty(200, dtype=torch.float32, device=DEV)
    ws = torch.empty(q.calibrate_workspace_bytes(p), dtype=torch.uint8, device=DEV)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    q.quantize(Wd, p, act, 0.3, q.DEFAULT_SIGN_SEED, c.cb, s_out, signs_out, sigma_out, packed, norm, ws, st)
    torch.cuda.synchronize()
    assert np.array_equal(s_out.cpu().numpy(), c.s) and np.array_equal(signs_out.cpu().numpy(), c.signs)
    assert np.array_equal(sigma_out.cpu().numpy(), c.sigma_gpu) and int(st.cpu()[0]) == 0
    # the Case encoded with the oracle's sigma; encode again with the GPU's own for the comparison
    packed2 = torch.empty_like(packed)
    norm2 = torch.empty_like(norm)
    q.encode(Wd, p, s_out, signs_out, sigma_out, c.cb, packed2, norm2)
    assert torch.equal(packed, packed2) and torch.equal(norm, norm2)
    # no scaling: chan_scale_out may be NULL
    q.quantize(Wd, p, None, 0.0, q.DEFAULT_SIGN_SEED, c.cb, None, signs_out, sigma_out, packed, norm, ws, st)
    q.calibrate(Wd, p, None, signs_out, sigma_out, ws, st)
    q.encode(Wd, p, None, signs_out, sigma_out, c.cb, packed2, norm2)
    assert torch.equal(packed, packed2) and torch.equal(norm, norm2)


@pytest.mark.parametrize("d_out,d_in", [(1, 8), (15, 1000), (16, 1024), (17, 2056), (100, 3072), (33, 8200)])
def test_distortion_sums_for_short_and_ragged_streams(orc, d_out, d_in):
    """The four sums of the distortion reduction (Corollaries 3 and 4) on bf16 pairs (W, W_hat) whose row
    streams are shorter than, equal to and longer than the copy ring, with columns that fill a thread
    tile only partly: single-matrix call and one batch of three copies against the oracle."""
    g = torch.Generator().manual_seed(d_out * 7919 + d_in)
    W = (torch.randn((d_out, d_in), generator=g) * torch.exp(torch.randn((d_out, 1), generator=g))).to(torch.bfloat16)
    What = (W.float() * (1 + 0.05 * torch.randn((d_out, d_in), generator=g))).to(torch.bfloat16)
    What[0, 0] = 0.0
    act = torch.exp(torch.randn(d_in, generator=g))
    ref = orc.distortion(_to_bits(W), _to_bits(What), act.numpy())
    Wd, Hd, ad = W.to(DEV), What.to(DEV), act.to(DEV)
    p = q.make_params(Wd, d_out, d_in, 2, 64)
    out4 = torch.full((4,), float("nan"), dtype=torch.float64, device=DEV)
    q.distortion(Wd, Hd, ad, p, out4)
    np.testing.assert_allclose(out4.cpu().numpy(), ref, rtol=1e-9)
    ref_plain = orc.distortion(_to_bits(W), _to_bits(What), None)
    q.distortion(Wd, Hd, None, p, out4)
    np.testing.assert_allclose(out4.cpu().numpy(), ref_plain, rtol=1e-9)
    # three matrices behind one batch handle: every one gets its own sums
    cb = _codebook(orc, 64)[1]
    dummy_b = torch.zeros(d_out * p.packed_row_stride + 64, dtype=torch.uint8, device=DEV)
    dummy_f = torch.ones(max(d_out, d_in), dtype=torch.float32, device=DEV)
    signs = torch.ones(d_in, dtype=torch.int8, device=DEV)
    dists = [torch.full((4,), float("nan"), dtype=torch.float64, device=DEV) for _ in range(3)]
    mats = [q.make_matrix(p, Wd, None, signs, dummy_f, ad, dummy_b, dummy_f, Hd, d) for d in dists]
    batch = q.Batch(mats, cb)
    batch.distortion()
    for d in dists:
        np.testing.assert_allclose(d.cpu().numpy(), ref, rtol=1e-9)


def test_batch_with_the_polar_quantiser(orc):
    """The batched phases take a polar codebook as they take a 2-D one: same bytes as the single-matrix
    calls (whose indices test_polar_baseline_codec checks against the oracle)."""
    Ba, Bp = 4, 4
    shapes = [(130, 2048), (33, 11776), (64, 512)]
    lv, _ = q.polar_train(Ba)
    cb = q.Codebook.polar(lv, Ba, Bp)
    _, a = _batch_problem(shapes, 256, 128, torch.bfloat16)
    _, b = _batch_problem(shapes, 256, 128, torch.bfloat16)
    st = torch.zeros(1, dtype=torch.int32, device=DEV)
    for s in a:
        ws = torch.empty(q.calibrate_workspace_bytes(s["p"]), dtype=torch.uint8, device=DEV)
        q.calibrate(s["W"], s["p"], s["s"], s["signs"], s["sigma"], ws, st)
        q.encode(s["W"], s["p"], s["s"], s["signs"], s["sigma"], cb, s["packed"], s["norm"], st)
        q.decode(s["packed"], s["norm"], s["s"], s["signs"], s["sigma"], cb, s["p"], s["what"])
    mats = [q.make_matrix(s["p"], s["W"], s["s"], s["signs"], s["sigma"], s["act"], s["packed"], s["norm"], s["what"],
                          s["dist"]) for s in b]
    batch = q.Batch(mats, cb)
    for x, y in zip(a, b):
        y["sigma"].copy_(x["sigma"])
    batch.encode(st)
    batch.decode()
    torch.cuda.synchronize()
    assert int(st.cpu()[0]) == 0
    for x, y in zip(a, b):
        assert torch.equal(x["packed"], y["packed"]) and torch.equal(x["norm"], y["norm"])
        assert torch.equal(x["what"].view(torch.int16), y["what"].view(torch.int16))
