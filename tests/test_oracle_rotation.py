"""Pins of the oracle's rotation, front half, calibration and small helpers.

Every expected value here comes from the paper (printed examples, Lemma 1 and
its remarks), from the mathematics (orthogonality, closed forms) or from a
library routine (numpy / torch) -- never from the CUDA path.
"""
import itertools
import os

import numpy as np
import pytest
import torch

from conftest import GOLDEN


def _read_small_hadamards():
    mats, cur, name = {}, [], None
    with open(os.path.join(GOLDEN, "hadamard_small.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            if line.startswith("H"):
                if name:
                    mats[name] = np.array(cur, np.float64)
                name, cur = line.strip(), []
            else:
                cur.append([int(t) for t in line.split()])
    mats[name] = np.array(cur, np.float64)
    return mats


def test_hadamard_by_hand(orc):
    """b = 2 and b = 4 written out by hand from the recursion (Appendix A.1, Definition 1)."""
    for name, H in _read_small_hadamards().items():
        b = H.shape[0]
        for q in range(b):
            e = np.zeros(b)
            e[q] = 1.0
            np.testing.assert_allclose(orc.hadamard_def(e), H[:, q] / np.sqrt(b), atol=1e-15)
        assert np.array_equal(orc.sylvester_matrix(b), H.astype(np.int8))


@pytest.mark.parametrize("b", [2, 8, 64, 128, 1024])
def test_sylvester_properties(orc, b):
    """H^T H = b I, H = H^T, and the popcount closed form equals the recursion (Definition 1)."""
    H = orc.sylvester_matrix(b).astype(np.float64)
    assert np.array_equal(H, H.T)
    assert np.array_equal(H.T @ H, b * np.eye(b))
    half = b // 2
    assert np.array_equal(H[:half, half:], H[:half, :half])
    assert np.array_equal(H[half:, half:], -H[:half, :half])
    rng = np.random.default_rng(b)
    v = rng.standard_normal(b)
    np.testing.assert_allclose(orc.hadamard_def(v), H @ v / np.sqrt(b), rtol=0, atol=1e-12)
    # butterfly (double and canonical f32) against the definition
    np.testing.assert_allclose(orc.fwht_f64(v), H @ v, rtol=0, atol=1e-11)
    v32 = v.astype(np.float32)
    np.testing.assert_allclose(orc.fwht_f32(v32), H @ v32.astype(np.float64), rtol=0,
                               atol=2e-6 * np.abs(v32).sum())


def test_fwht_f32_is_exact_on_integers(orc):
    """Small integers are exact in f32, so the canonical butterfly must equal H v exactly."""
    rng = np.random.default_rng(3)
    v = rng.integers(-100, 100, 256).astype(np.float32)
    H = orc.sylvester_matrix(256).astype(np.float64)
    assert np.array_equal(orc.fwht_f32(v).astype(np.float64), H @ v.astype(np.float64))


def _matrix_of(fn, d):
    return np.stack([fn(np.eye(d)[:, j]) for j in range(d)], axis=1)


@pytest.mark.parametrize("d_in,b", [(8, 4), (64, 16), (256, 128)])
def test_lemma1_isometry(orc, d_in, b):
    """Lemma 1: R_fwd = F S and R_inv = S F are orthogonal and mutually inverse; the remark
    after it: they are different matrices when the mask is not trivial."""
    signs = orc.make_signs(12345, d_in)
    assert set(np.unique(signs)) == {-1, 1}
    Rf = _matrix_of(lambda e: orc.rotate_fwd(e, signs, b), d_in)
    Ri = _matrix_of(lambda e: orc.rotate_inv(e, signs, b), d_in)
    I = np.eye(d_in)
    np.testing.assert_allclose(Rf.T @ Rf, I, atol=1e-12)
    np.testing.assert_allclose(Ri.T @ Ri, I, atol=1e-12)
    np.testing.assert_allclose(Ri @ Rf, I, atol=1e-12)
    H = orc.sylvester_matrix(b).astype(np.float64) / np.sqrt(b)
    F = np.kron(np.eye(d_in // b), H)
    S = np.diag(signs.astype(np.float64))
    np.testing.assert_allclose(Rf, F @ S, atol=1e-12)  # signs BEFORE the transform on encode
    np.testing.assert_allclose(Ri, S @ F, atol=1e-12)  # signs AFTER the transform on decode
    assert np.abs(Rf - Ri).max() > 0.1  # not an involution
    assert np.abs(Rf - Rf.T).max() > 0.1  # not symmetric
    # norms, distances, inner products and per-block energy
    rng = np.random.default_rng(7)
    u, v = rng.standard_normal(d_in), rng.standard_normal(d_in)
    yu, yv = orc.rotate_fwd(u, signs, b), orc.rotate_fwd(v, signs, b)
    assert abs(np.linalg.norm(yu) - np.linalg.norm(u)) < 1e-12
    assert abs(np.linalg.norm(yu - yv) - np.linalg.norm(u - v)) < 1e-12
    assert abs(yu @ yv - u @ v) < 1e-12
    np.testing.assert_allclose((yu.reshape(-1, b) ** 2).sum(1), (u.reshape(-1, b) ** 2).sum(1), rtol=1e-12)
    np.testing.assert_allclose(orc.rotate_inv(yu, signs, b), u, atol=1e-12)


def test_energy_spreading_exact_over_all_masks(orc):
    """Remark after Lemma 1: E_S[(R v)_j] = 0 and E_S[(R v)_j^2] = |v_block|^2 / b for
    Rademacher signs; averaged over all 2^8 masks of one b = 8 block this is exact."""
    b = 8
    rng = np.random.default_rng(11)
    v = rng.standard_normal(b)
    m1, m2 = np.zeros(b), np.zeros(b)
    for mask in itertools.product([-1, 1], repeat=b):
        y = orc.rotate_fwd(v, np.array(mask, np.int8), b)
        m1 += y
        m2 += y * y
    np.testing.assert_allclose(m1 / 2**b, 0, atol=1e-13)
    np.testing.assert_allclose(m2 / 2**b, (v @ v) / b, rtol=1e-12)


def test_sign_generator_spec(orc):
    """Repository specification of the mask (the paper fixes only 'a fixed 64-bit seed'):
    top bit of the SplitMix64 finaliser of seed + (j+1)*golden.  Checked against a
    pure-Python big-integer evaluation."""
    M = 2**64 - 1

    def mix(x):
        x ^= x >> 30
        x = (x * 0xBF58476D1CE4E5B9) & M
        x ^= x >> 27
        x = (x * 0x94D049BB133111EB) & M
        x ^= x >> 31
        return x

    for seed in (0, 1, 0xDEADBEEFCAFEF00D):
        s = orc.make_signs(seed, 300)
        want = [-1 if mix((seed + 0x9E3779B97F4A7C15 * (j + 1)) & M) >> 63 else 1 for j in range(300)]
        assert s.tolist() == want
    big = orc.make_signs(2024, 1 << 16).astype(np.float64)
    assert abs(big.mean()) < 4 / np.sqrt(big.size)  # balanced
    assert abs(np.mean(big[1:] * big[:-1])) < 4 / np.sqrt(big.size)  # no lag-1 correlation


def test_block_size_rule_printed_examples(orc):
    with open(os.path.join(GOLDEN, "block_rule.txt")) as f:
        rows = [l.split() for l in f if not l.startswith("#") and l.strip()]
    for d_in, b in rows:
        assert orc.block_size_rule(int(d_in)) == int(b)
    assert orc.block_size_rule(4096) == 1024 and orc.block_size_rule(11008) == 256
    assert orc.block_size_rule(6) == 2 and orc.block_size_rule(7) == 1


def test_bpw_printed_values(orc):
    """Section 3.7 closed form, pooled over the MLP matrices, reproduces the printed bitrates."""
    assert abs(orc.bpw(1, 2048, 2048, False) - 5.5078125) < 1e-12  # "approximately 5.51 bpw"
    assert abs(orc.bpw(1, 2048, 128, False) - 3.5078125) < 1e-12  # "bpw ~ 3.51" (Section 3.8)
    with open(os.path.join(GOLDEN, "bpw_printed.txt")) as f:
        rows = [l.split() for l in f if not l.startswith("#") and l.strip()]
    for label, hidden, inter, B, has_s, printed, digits, *_ in rows:
        hidden, inter, B, has_s, digits = int(hidden), int(inter), int(B), int(has_s), int(digits)
        mats = [(inter, hidden), (inter, hidden), (hidden, inter)]  # gate, up, down
        bits = sum(orc.bpw(o, i, 2**B, bool(has_s)) * o * i for o, i in mats)
        pooled = bits / sum(o * i for o, i in mats)
        assert abs(pooled - float(printed)) <= 0.5 * 10**-digits + 1e-9, (label, pooled, printed)


def test_packed_row_bytes(orc):
    assert orc.packed_row_bytes(2048, 2048) == 1408  # 1024 pairs x 11 bits, no padding
    assert orc.packed_row_bytes(5120, 2048) == 3520
    assert orc.packed_row_bytes(6, 8) == 2  # 9 bits -> 2 bytes


def test_packing_hand_worked_and_roundtrip(orc):
    with open(os.path.join(GOLDEN, "packing_example.txt")) as f:
        rows = [l.split("|") for l in f if not l.startswith("#") and l.strip()]
    for B, idx, want in rows:
        idx = [int(t, 16) for t in idx.split()]
        want = bytes(int(t, 16) for t in want.split())
        got = orc.pack_row(np.array(idx, np.int32), int(B), len(want))
        assert bytes(got) == want
        assert orc.unpack_row(got, len(idx), int(B)).tolist() == idx
    rng = np.random.default_rng(5)
    for B in range(1, 13):
        idx = rng.integers(0, 2**B, 257).astype(np.int32)
        p = orc.pack_row(idx, B)
        assert p.size == (257 * B + 7) // 8
        assert np.array_equal(orc.unpack_row(p, 257, B), idx)
        # the same stream through Python big integers
        big = sum(int(v) << (k * B) for k, v in enumerate(idx))
        assert bytes(p) == big.to_bytes(p.size, "little")


def test_bf16_rounding(orc):
    """One rounding double -> bf16, ties to even.  On f32-representable inputs it must agree
    with torch's f32 -> bf16 conversion; the double-rounding trap 1 + 2^-8 + 2^-30 must round up."""
    rng = np.random.default_rng(9)
    x = np.concatenate([rng.standard_normal(4000) * 10.0 ** rng.integers(-30, 30, 4000),
                        [0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895e38, 3.4e38, 1e-40, 9.2e-41, 4.5e-41]])
    x = x.astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = orc.f64_to_bf16(x.astype(np.float64))
    assert np.array_equal(got, want)
    assert int(orc.f64_to_bf16(1.0 + 2.0**-8 + 2.0**-30)[0]) == 0x3F81
    assert int(orc.f64_to_bf16(1.0 + 2.0**-8)[0]) == 0x3F80  # exact tie -> even


def test_channel_scales(orc):
    """Section B.2: s_j ~ r_j^alpha, geometric mean one, clamp [1/16, 16]."""
    rng = np.random.default_rng(21)
    r = np.exp(rng.standard_normal(512)).astype(np.float32)
    assert np.array_equal(orc.channel_scales(r, 0.0), np.ones(512, np.float32))
    for alpha in (0.3, 0.5, 0.8):
        s = orc.channel_scales(r, alpha).astype(np.float64)
        assert abs(np.log(s).mean()) < 1e-6  # geometric mean 1 (no clamp hit here)
        ratio = s / r.astype(np.float64) ** alpha  # proportional to r^alpha
        np.testing.assert_allclose(ratio, ratio[0], rtol=1e-6)
        assert np.all(np.diff(s[np.argsort(r)]) >= 0)  # monotone in r_j
    r2 = r.copy()
    r2[:4] = [1e-30, 0.0, 1e30, 1e12]
    s = orc.channel_scales(r2, 0.8)
    assert s.min() == np.float32(1 / 16) and s.max() == np.float32(16)
    assert s[0] == s[1] == np.float32(1 / 16) and s[2] == np.float32(16)
    # clamp happens after normalisation, without re-normalising the rest
    t = 0.8 * np.log(np.maximum(r2.astype(np.float64), np.finfo(np.float32).tiny))
    want = np.clip(np.exp(t - t.mean()), 1 / 16, 16)
    np.testing.assert_allclose(s, want, rtol=1e-6)


def _rows(rng, d_out, d_in, dtype):
    W = (rng.standard_t(4, (d_out, d_in)) * np.exp(0.7 * rng.standard_normal((d_out, 1)))).astype(np.float32)
    if dtype == "bf16":
        return torch.from_numpy(W).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    return W


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("d_in,b", [(256, 64), (512, 128), (2048, 1024)])
def test_canonical_path_matches_definition(orc, dtype, d_in, b):
    """The canonical f32 path equals the double definition (scale -> norm -> F S u) within
    1e-5 relative, normwise per block, and its row norm within 1e-6; textbook ||.||_2."""
    rng = np.random.default_rng(d_in + b)
    W = _rows(rng, 6, d_in, dtype)
    s = orc.channel_scales(np.exp(rng.standard_normal(d_in)).astype(np.float32), 0.5)
    signs = orc.make_signs(99, d_in)
    for i in range(W.shape[0]):
        y32, r32, rc = orc.front_row(W[i], b, s, signs)
        y64, r64, rc2 = orc.front_row_def(W[i], b, s, signs)
        assert rc == 0 and rc2 == 0
        wf = orc.bf16_to_f32(W[i]).astype(np.float64) if dtype == "bf16" else W[i].astype(np.float64)
        assert abs(r64 - np.linalg.norm(wf * s.astype(np.float64))) <= 1e-12 * r64
        assert abs(float(r32) - r64) <= 1e-6 * r64
        assert abs(np.linalg.norm(y64) - 1.0) < 1e-12  # unit direction, isometry
        err = np.abs(y32.astype(np.float64) - y64).reshape(-1, b).max(1)
        ref = np.abs(y64).reshape(-1, b).max(1)
        assert np.all(err <= 1e-5 * ref)


def test_front_row_special_cases(orc):
    d_in, b = 128, 32
    signs = orc.make_signs(1, d_in)
    y, r, rc = orc.front_row(np.zeros(d_in, np.float32), b, None, signs)
    assert rc == 0 and r == 0 and not y.any()  # zero row -> zero direction
    w = np.zeros(d_in, np.float32)
    w[5] = np.inf
    assert orc.front_row(w, b, None, signs)[2] == orc.ORC_ERR_NONFINITE
    w[5] = np.nan
    assert orc.front_row(w, b, None, signs)[2] == orc.ORC_ERR_NONFINITE
    # a unit vector maps to a signed, scaled column of H_b inside its block only
    w = np.zeros(d_in, np.float32)
    w[37] = -3.0
    y, r, rc = orc.front_row(w, b, None, signs)
    H = orc.sylvester_matrix(b).astype(np.float64)
    want = np.zeros(d_in)
    want[32:64] = -signs[37] * H[:, 5] / np.sqrt(b)
    assert r == 3.0
    np.testing.assert_allclose(y, want, atol=1e-7)


def test_calibration_recovers_sigma(orc):
    """Section 3.4: for circular-Gaussian pairs E|z_k| = sigma_k sqrt(pi/2).  Rows are built
    as R_inv applied to pairs with known sigma_k (sum of 2 sigma_k^2 = 1, so rows have unit norm
    up to O(d^-1/2)); the estimate converges at rate n^-1/2 with n = 1024 rows."""
    d_in, b, n_rows = 1024, 128, 2048  # only 1024 of the 2048 rows may be used
    rng = np.random.default_rng(31)
    sig = np.exp(0.5 * rng.standard_normal(d_in // 2))
    sig /= np.sqrt(2 * (sig**2).sum())
    signs = orc.make_signs(4, d_in)
    Y = rng.standard_normal((n_rows, d_in)) * np.repeat(sig, 2)
    W = np.stack([orc.rotate_inv(y, signs, b) for y in Y]).astype(np.float32)
    got, rc = orc.calibrate(W, b, None, signs)
    assert rc == 0
    ratio = got.astype(np.float64) / sig
    assert abs(ratio.mean() - 1.0) < 5e-3
    assert ratio.std() < 2.5 * 0.5227 / np.sqrt(1024)  # Rayleigh cv = sqrt(4/pi - 1) = 0.5227
    # the documented row subset: rows floor(t * d_out / n); a direct numpy evaluation on it
    rows = (np.arange(1024) * n_rows) // 1024
    amp = np.zeros(d_in // 2)
    for i in rows:
        y, r, _ = orc.front_row(W[i], b, None, signs)
        amp += np.hypot(y[0::2].astype(np.float64), y[1::2].astype(np.float64))
    np.testing.assert_allclose(got, amp / 1024 / np.sqrt(np.pi / 2), rtol=1e-6)


def test_calibration_edge_cases(orc):
    d_in, b = 64, 16
    signs = orc.make_signs(4, d_in)
    sig, rc = orc.calibrate(np.zeros((5, d_in), np.float32), b, None, signs)
    assert rc == 0
    np.testing.assert_allclose(sig, 1 / np.sqrt(d_in), rtol=1e-7)  # no usable row
    W = np.zeros((3, d_in), np.float32)
    W[1, :16] = 1.0  # energy in one block only: other pairs hit the floor
    sig, rc = orc.calibrate(W, b, None, signs)
    assert np.all(sig[8:] == np.float32(1e-4 / np.sqrt(d_in)))
    assert np.all(sig[:8] > 0.01)
