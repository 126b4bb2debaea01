"""CPU-only checks of libqamw.so: the shared library loads and exports every symbol that
include/qamw.h declares, its host-side helpers agree with the oracle, the exact search table
returns what an exhaustive scan returns, and argument errors are reported before anything is
launched.  No compute call needs a GPU here."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from conftest import ROOT, load_golden_codebook
from paper_2605_26339_b200 import binding as q


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "qamw.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(qamw_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_functions()
    assert len(names) >= 19 and "qamw_encode" in names and "qamw_calibrate_static" in names
    lib = q.lib()
    for n in names:
        assert getattr(lib, n) is not None, n
    assert sorted(q.EXPORTED) == names  # the binding's own list is complete too


def test_helpers_agree_with_oracle(orc):
    for seed, d_in in [(q.DEFAULT_SIGN_SEED, 4096), (1, 130), (2**64 - 1, 64)]:
        assert np.array_equal(q.make_signs(seed, d_in), orc.make_signs(seed, d_in))
    rng = np.random.default_rng(0)
    act = np.exp(rng.standard_normal(1000)).astype(np.float32)
    act[::97] *= 20
    act[5] = 0.0
    for alpha in (0.0, 0.3, 0.5, 0.8):
        a = q.channel_scales(act, alpha)
        b = orc.channel_scales(act, float(np.float32(alpha)))
        assert np.all(np.abs(a.view(np.int32) - b.view(np.int32)) <= 1)  # same formula, libm may differ by an ulp
    for d_in in (2048, 5632, 5120, 13824, 4096, 11008, 6, 1, 1024 * 3):
        assert q.block_size_rule(d_in) == orc.block_size_rule(d_in)
    for d_in in (2, 6, 128, 5120, 13824):
        for K in (2, 64, 128, 256, 2048, 4096):
            assert q.packed_row_bytes(d_in, K) == orc.packed_row_bytes(d_in, K)
            assert q.bpw(4096, d_in, K, True) == pytest.approx(orc.bpw(4096, d_in, K, True), abs=1e-15)
    assert q.status_to_error(0) == 0 and q.status_to_error(1) == q.ERR_NONFINITE


@pytest.mark.parametrize("K", [16, 64])
def test_library_trainer_is_a_lloyd_fixed_point_like_the_oracles(orc, K):
    """The library's trainer follows the same written recipe as the oracle's (same samples, same
    initialisation) but sums in chunks, so codewords may differ in the last bits: compare quality and
    check the Lloyd conditions with the oracle's own routines."""
    n = 1 << 14
    cb, mse = q.train_codebook(K, n, 3, 500, 0.0)
    cb_o, mse_o, _ = orc.train_codebook(K, n, 3, 500, 0.0)
    assert abs(mse - mse_o) <= 2e-3 * mse_o
    z = orc.gauss_pairs(3, n)
    assign, mse2 = orc.lloyd_assign(z, cb.astype(np.float64))
    assert abs(mse2 - mse) < 1e-12
    for k in range(K):  # centroid condition up to the f32 rounding of the stored codebook
        if np.any(assign == k):  # a cell that lost all its samples keeps its codeword
            np.testing.assert_allclose(cb[k], z[assign == k].mean(0), atol=2e-6)
    assert np.bincount(assign, minlength=K).min() >= 0 and (np.bincount(assign, minlength=K) > 0).sum() >= K - 2
    r2 = (cb.astype(np.float64) ** 2).sum(1)
    assert np.all(np.diff(r2) >= 0)  # sorted by radius


def _columns(cmap, grid, z, nudge=0.0):
    """The cell map of include/qamw.h in f32 steps (numpy has no fused multiply-add: a product and a sum
    rounded separately land, at worst, in the neighbouring column, whose list holds the answer too).
    `nudge` moves the value by a fraction of a column before the rounding."""
    zmax, c0, c1, c2 = (np.float32(v) for v in cmap)
    c = np.minimum(np.maximum(z.astype(np.float32), -zmax), zmax)
    t = c * c
    u = c * (c0 + t * (c1 + t * c2))
    col = np.rint(u.astype(np.float64) + nudge).astype(np.int64) + (grid - 1) // 2
    return np.clip(col, 0, grid - 1)


def _table_search(cb, cmap, cells, ovf, grid, z, nudge=0.0):
    """What the device's table search computes, in numpy (f32 cell arithmetic, f64 distances)."""
    col = _columns(cmap, grid, z, nudge)
    rec = cells[col[:, 1] * grid + col[:, 0]]
    out = np.empty(len(z), np.int64)
    for i in range(len(z)):
        r = rec[i]
        cand = ovf[r[1]: r[1] + r[2]] if r[0] == 0xFFFF else r
        c = cb[cand.astype(np.int64)].astype(np.float64)
        d = ((z[i].astype(np.float64) - c) ** 2).sum(1)
        out[i] = cand[int(np.argmin(d))]
    return out


@pytest.mark.parametrize("K,grid", [(64, 0), (256, 0), (2048, 0), (2048, 41), (4096, 0)])
def test_search_table_is_exact(K, grid):
    """Every cell lists all codewords whose nearest-neighbour region meets it: scanning the list
    gives the exhaustive answer, for Gaussian points, heavy tails and points far outside."""
    cb = load_golden_codebook(K)
    cmap, cells, ovf, info = q.search_table_build(cb, grid, 1 << 20)
    g = int(info[0])
    assert g % 2 == 1 and cells.shape == (g * g, 4) and int(info[5]) == cells.size * 2 + int(info[4]) * 2
    assert int(info[5]) % 16 == 0  # the device copies it in 16-byte pieces
    rng = np.random.default_rng(K + grid)
    z = np.concatenate([rng.standard_normal((6000, 2)), 3 * rng.standard_t(3, (3000, 2)),
                        rng.uniform(-9, 9, (2000, 2)), 1000 * rng.standard_normal((500, 2)),
                        cb[:64].astype(np.float64) + 1e-4 * rng.standard_normal((64, 2))]).astype(np.float32)
    z = z[np.abs(z).max(1) < 16000]
    d = ((z[:, None, :].astype(np.float64) - cb[None].astype(np.float64)) ** 2).sum(2)
    best = d.argmin(1)
    part = np.partition(d, 1, axis=1)
    near_tie = (part[:, 1] - part[:, 0]) < 1e-6 * part[:, 1]
    # the lists also cover a point that rounding carries into the neighbouring column or row
    for nudge in (0.0, 1 / 512, -1 / 512):
        got = _table_search(cb, cmap, cells, ovf, g, z, nudge)
        assert np.all((got == best) | near_tie)


def test_default_table_fits_the_encoder_and_explicit_grid_is_honoured():
    cb = load_golden_codebook(2048)
    _, _, _, info = q.search_table_build(cb, 0, 77 * 1024)
    assert info[5] <= 77 * 1024 and info[2] >= 4  # longest list beyond 4: overflow lists exist
    _, cells, _, info = q.search_table_build(cb, 25, 1 << 20)
    assert info[0] == 25 and cells.shape[0] == 625
    with pytest.raises(q.QamwError) as e:
        q.search_table_build(cb, 201, 64 * 1024)
    assert e.value.code == q.ERR_NOMEM
    with pytest.raises(q.QamwError) as e:
        q.search_table_build(cb, 24, 1 << 20)  # the grid side is odd
    assert e.value.code == q.ERR_ARG


def test_cell_map_is_increasing_and_stays_inside_the_grid():
    cb = load_golden_codebook(256)
    for grid in (3, 25, 99, 255):
        cmap, _, _, info = q.search_table_build(cb, grid, 1 << 22)
        z = np.linspace(-float(cmap[0]) * 1.5, float(cmap[0]) * 1.5, 20001).astype(np.float32)
        zz = np.stack([z, z], 1)
        col = _columns(cmap, grid, zz)[:, 0]
        assert np.all(np.diff(col) >= 0) and col.min() == 0 and col.max() == grid - 1
        assert np.all(np.diff(col) <= 1)  # no column is skipped at this sampling density
        far = np.array([[-1e30, 1e30], [np.inf, -np.inf]], np.float32)
        assert _columns(cmap, grid, far).tolist() == [[0, grid - 1], [grid - 1, 0]]


def test_argument_errors_are_reported_before_any_launch():
    lib = q.lib()
    dummy = (C.c_char * 64)()
    ptr = C.cast(dummy, C.c_void_p)

    def params(**kw):
        base = dict(d_out=4, d_in=256, block=64, K=256, w_dtype=q.DTYPE_BF16, flags=0, w_row_stride=256,
                    packed_row_stride=128)
        base.update(kw)
        return q.Params(**base)

    def enc(p, W=ptr, cb=ptr):
        return lib.qamw_encode(W, C.byref(p), None, ptr, ptr, cb, ptr, ptr, None, None)

    assert enc(params(d_in=255, w_row_stride=255)) == q.ERR_SHAPE            # odd row length
    assert enc(params(block=96)) == q.ERR_SHAPE                              # block not a power of two
    assert enc(params(block=128, d_in=192, w_row_stride=192)) == q.ERR_SHAPE  # block does not divide d_in
    assert enc(params(K=3)) == q.ERR_SHAPE
    assert enc(params(K=8192)) == q.ERR_SHAPE
    assert enc(params(block=2048, d_in=4096, w_row_stride=4096)) == q.ERR_SHAPE
    assert enc(params(d_in=32768, block=128, w_row_stride=32768)) == q.ERR_SHAPE  # longer than a block can hold
    assert enc(params(w_dtype=7)) == q.ERR_ARG
    assert enc(params(w_row_stride=100)) == q.ERR_ARG
    assert enc(params(), W=None) == q.ERR_ARG
    assert enc(params(), cb=None) == q.ERR_ARG
    assert lib.qamw_decode(None, ptr, None, ptr, ptr, ptr, C.byref(params()), ptr, None) == q.ERR_ARG
    assert lib.qamw_distortion(ptr, None, None, C.byref(params()), ptr, None) == q.ERR_ARG
    assert lib.qamw_calibrate(ptr, C.byref(params()), None, ptr, ptr, None, 0, None, None) == q.ERR_ARG
    assert lib.qamw_calibrate_static(ptr, C.byref(params(block=96)), None, ptr, ptr, None, None) == q.ERR_SHAPE
    assert lib.qamw_rotate(ptr, None, None, ptr, ptr, ptr, None, None) == q.ERR_ARG
    # the one-call form checks its arguments before touching the device
    assert lib.qamw_quantize(None, C.byref(params()), None, 0.0, 1, ptr, None, ptr, ptr, ptr, ptr, ptr, 1 << 20, None, None) == q.ERR_ARG
    assert lib.qamw_quantize(ptr, C.byref(params(block=96)), None, 0.0, 1, ptr, None, ptr, ptr, ptr, ptr, ptr, 1 << 20, None, None) == q.ERR_SHAPE
    act = np.ones(256, np.float32)
    assert lib.qamw_quantize(ptr, C.byref(params()), act.ctypes.data, 0.3, 1, ptr, None, ptr, ptr, ptr, ptr, ptr, 1 << 20, None, None) == q.ERR_ARG  # scaling without a place for the scales
    assert lib.qamw_quantize(ptr, C.byref(params()), None, 0.0, 1, ptr, None, ptr, ptr, ptr, ptr, ptr, 8, None, None) == q.ERR_NOMEM
    assert lib.qamw_round_f16(None, 4, None) == q.ERR_ARG and lib.qamw_round_f16(None, 0, None) == q.QAMW_OK
    assert lib.qamw_renorm_row_norms(None, ptr, ptr, ptr, C.byref(params()), ptr, None) == q.ERR_ARG
    # batches: argument checks come before any CUDA call
    hb = C.c_void_p()
    item = q.Matrix(params(block=96), ptr.value, None, ptr.value, ptr.value, None, ptr.value, ptr.value, ptr.value, ptr.value)
    arr = (q.Matrix * 1)(item)
    assert lib.qamw_batch_create(None, 1, ptr, C.byref(hb)) == q.ERR_ARG
    assert lib.qamw_batch_create(arr, 0, ptr, C.byref(hb)) == q.ERR_ARG
    assert lib.qamw_batch_create(arr, 1, None, C.byref(hb)) == q.ERR_ARG
    assert lib.qamw_batch_create(arr, 1, ptr, C.byref(hb)) == q.ERR_SHAPE  # block is not a power of two
    assert lib.qamw_encode_batch(None, None, None) == q.ERR_ARG
    assert lib.qamw_decode_batch(None, None) == q.ERR_ARG
    assert lib.qamw_distortion_batch(None, None) == q.ERR_ARG
    assert lib.qamw_calibrate_batch(None, ptr, 64, None, None) == q.ERR_ARG
    assert lib.qamw_batch_workspace_bytes(None) == 0
    h = C.c_void_p()
    cbk = np.zeros((4, 2), np.float32)
    assert lib.qamw_codebook_create(cbk.ctypes.data, 3, 0, C.byref(h)) == q.ERR_SHAPE
    assert lib.qamw_codebook_create(None, 4, 0, C.byref(h)) == q.ERR_ARG
    # sizes reported without touching the device
    assert q.calibrate_workspace_bytes(params(d_out=5120, d_in=5120, block=128, w_row_stride=5120,
                                              packed_row_stride=3520)) <= q.STATIC_SCRATCH_BYTES
    assert q.calibrate_workspace_bytes(params(block=96)) == 0
    assert q.packed_row_bytes(255, 256) == 0 and q.block_size_rule(0) == 0
    with pytest.raises(q.QamwError):
        q.make_signs(1, 0)


@pytest.mark.parametrize("Ba", [0, 1, 3, 5])
def test_polar_levels_and_table_agree_with_oracle(orc, Ba):
    """The library's Rayleigh Lloyd-Max levels (closed-form moments) against the oracle's (Simpson
    quadrature): two implementations of Section 3.5's amplitude quantiser.  Lloyd's iteration creeps
    towards its fixed point, so the levels agree to the stopping tolerances and the distortion, which
    is flat there, far more closely.  Given the same levels the reconstruction tables are identical."""
    lv, c = q.polar_train(Ba)
    lo, co = orc.rayleigh_lloyd_max(1 << Ba)
    assert np.allclose(lv, lo, atol=1e-5) and abs(c - co) < 1e-9
    assert np.array_equal(q.polar_codebook(lv, Ba, 4), orc.polar_codebook(lv, Ba, 4))
    lib = q.lib()
    h = C.c_void_p()
    assert lib.qamw_polar_train(13, lv.ctypes.data, None) == q.ERR_SHAPE
    assert lib.qamw_polar_train(2, None, None) == q.ERR_ARG
    assert lib.qamw_polar_codebook(lv.ctypes.data, 7, 6, lv.ctypes.data) == q.ERR_SHAPE  # more than 4096 points
    assert lib.qamw_codebook_create_polar(None, 2, 2, C.byref(h)) == q.ERR_ARG
    bad = np.array([1.0, 0.5], np.float32)  # not ascending
    assert lib.qamw_codebook_create_polar(bad.ctypes.data, 1, 2, C.byref(h)) == q.ERR_ARG
