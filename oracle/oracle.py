"""ctypes front end of the plain-C QAM-W oracle (``qamw_oracle.c``).

TEST INFRASTRUCTURE ONLY: the test-suite, the smoke check and the benchmark's
cpu-baseline / reference arm are the only callers.  Nothing here touches the
CUDA library, and the CUDA library never imports this module.

All arrays are numpy; weights are either float32 or bf16 bit patterns held in a
``uint16`` array (``w_dtype`` 0 / 1).
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "qamw_oracle.c")
_OUT_DIR = os.path.join(_HERE, "_build")
_LIB_PATH = os.path.join(_OUT_DIR, "libqamw_oracle.so")
_lock = threading.Lock()
_lib = None

ORC_OK = 0
ORC_ERR_ARG = -1
ORC_ERR_NONFINITE = -5


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict IEEE: no contraction, no fast-math)."""
    os.makedirs(_OUT_DIR, exist_ok=True)
    if (not force and os.path.exists(_LIB_PATH)
            and os.path.getmtime(_LIB_PATH) >= os.path.getmtime(_SRC)):
        return _LIB_PATH
    tmp = _LIB_PATH + f".tmp{os.getpid()}"
    cmd = ["gcc", "-std=c11", "-O2", "-fPIC", "-shared", "-fopenmp", "-ffp-contract=off",
           "-fno-fast-math", "-Wall", "-Wextra", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB_PATH)
    return _LIB_PATH


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            L.orc_mix64.restype = C.c_uint64
            L.orc_mix64.argtypes = [C.c_uint64]
            L.orc_packed_row_bytes.restype = C.c_int64
            L.orc_bpw.restype = C.c_double
            L.orc_lloyd_assign.restype = C.c_double
            L.orc_codebook_mse.restype = C.c_double
            L.orc_f64_to_bf16.restype = C.c_uint16
            L.orc_f64_to_bf16.argtypes = [C.c_double]
            _lib = L
    return _lib


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _c(a, dtype):
    return None if a is None else np.ascontiguousarray(a, dtype=dtype)


def _w_dtype(W):
    if W.dtype == np.float32:
        return 0
    if W.dtype == np.uint16:
        return 1
    raise TypeError("W must be float32 or uint16 (bf16 bits)")


def num_threads() -> int:
    return int(lib().orc_num_threads())


def mix64(x: int) -> int:
    return int(lib().orc_mix64(C.c_uint64(x & (2**64 - 1))))


def make_signs(seed: int, d_in: int) -> np.ndarray:
    out = np.empty(d_in, np.int8)
    lib().orc_make_signs(C.c_uint64(seed), C.c_int(d_in), _p(out))
    return out


def gauss_pairs(seed: int, n: int) -> np.ndarray:
    out = np.empty((n, 2), np.float64)
    lib().orc_gauss_pairs(C.c_uint64(seed), C.c_uint64(n), _p(out))
    return out


def block_size_rule(d_in: int) -> int:
    return int(lib().orc_block_size_rule(C.c_int(d_in)))


def packed_row_bytes(d_in: int, K: int) -> int:
    return int(lib().orc_packed_row_bytes(C.c_int(d_in), C.c_int(K)))


def bpw(d_out: int, d_in: int, K: int, has_channel_scales: bool) -> float:
    return float(lib().orc_bpw(C.c_int(d_out), C.c_int(d_in), C.c_int(K), C.c_int(int(has_channel_scales))))


def channel_scales(act_rms: np.ndarray, alpha: float) -> np.ndarray:
    r = _c(act_rms, np.float32)
    out = np.empty(r.shape[0], np.float32)
    lib().orc_channel_scales(_p(r), C.c_int(r.shape[0]), C.c_double(alpha), _p(out))
    return out


def f64_to_bf16(v) -> np.ndarray:
    v = np.atleast_1d(np.asarray(v, np.float64))
    L = lib()
    return np.array([L.orc_f64_to_bf16(C.c_double(x)) for x in v.ravel()], np.uint16).reshape(v.shape)


def bf16_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.asarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32)


def hadamard_def(v: np.ndarray) -> np.ndarray:
    v = _c(v, np.float64)
    out = np.empty_like(v)
    lib().orc_hadamard_def(_p(v), C.c_int(v.shape[0]), _p(out))
    return out


def sylvester_matrix(b: int) -> np.ndarray:
    H = np.zeros((b, b), np.int8)
    lib().orc_sylvester_matrix(C.c_int(b), _p(H))
    return H


def rotate_fwd(u, signs, b) -> np.ndarray:
    u = _c(u, np.float64)
    s = _c(signs, np.int8)
    y = np.empty_like(u)
    lib().orc_rotate_fwd(_p(u), _p(s), C.c_int(u.shape[0]), C.c_int(b), _p(y))
    return y


def rotate_inv(y, signs, b) -> np.ndarray:
    y = _c(y, np.float64)
    s = _c(signs, np.int8)
    u = np.empty_like(y)
    lib().orc_rotate_inv(_p(y), _p(s), C.c_int(y.shape[0]), C.c_int(b), _p(u))
    return u


def fwht_f32(x: np.ndarray) -> np.ndarray:
    x = np.array(x, np.float32, copy=True)
    lib().orc_fwht_f32(_p(x), C.c_int(x.shape[0]))
    return x


def fwht_f64(x: np.ndarray) -> np.ndarray:
    x = np.array(x, np.float64, copy=True)
    lib().orc_fwht_f64(_p(x), C.c_int(x.shape[0]))
    return x


def front_row(w_row, b, chan_scale, signs):
    """Canonical f32 path for one row -> (y f32[d_in], r f32, status)."""
    w = np.ascontiguousarray(w_row)
    d_in = w.shape[0]
    y = np.empty(d_in, np.float32)
    r = C.c_float(0)
    rc = lib().orc_front_row(_p(w), C.c_int(_w_dtype(w)), C.c_int(d_in), C.c_int(b),
                             _p(_c(chan_scale, np.float32)), _p(_c(signs, np.int8)), _p(y), C.byref(r))
    return y, np.float32(r.value), int(rc)


def front_row_def(w_row, b, chan_scale, signs):
    """Definition path (double, O(b^2) Hadamard) for one row -> (y f64, r f64, status)."""
    w = np.ascontiguousarray(w_row)
    d_in = w.shape[0]
    y = np.empty(d_in, np.float64)
    r = C.c_double(0)
    rc = lib().orc_front_row_def(_p(w), C.c_int(_w_dtype(w)), C.c_int(d_in), C.c_int(b),
                                 _p(_c(chan_scale, np.float32)), _p(_c(signs, np.int8)), _p(y), C.byref(r))
    return y, float(r.value), int(rc)


def calibrate(W, b, chan_scale, signs):
    W = np.ascontiguousarray(W)
    d_out, d_in = W.shape
    sigma = np.empty(d_in // 2, np.float32)
    rc = lib().orc_calibrate(_p(W), C.c_int(_w_dtype(W)), C.c_int(d_out), C.c_int(d_in), C.c_int64(d_in),
                             C.c_int(b), _p(_c(chan_scale, np.float32)), _p(_c(signs, np.int8)), _p(sigma))
    return sigma, int(rc)


def nearest(z, codebook):
    """Exhaustive search for each 2-D point of z[n,2] -> (idx, best d2, second d2)."""
    z = _c(z, np.float64).reshape(-1, 2)
    cb = _c(codebook, np.float32)
    K = cb.shape[0]
    idx = np.empty(z.shape[0], np.int32)
    d1 = np.empty(z.shape[0], np.float64)
    d2 = np.empty(z.shape[0], np.float64)
    L = lib()
    L.orc_nearest.restype = C.c_int
    b1, b2 = C.c_double(), C.c_double()
    for i in range(z.shape[0]):
        idx[i] = L.orc_nearest(C.c_double(z[i, 0]), C.c_double(z[i, 1]), _p(cb), C.c_int(K),
                               C.byref(b1), C.byref(b2))
        d1[i], d2[i] = b1.value, b2.value
    return idx, d1, d2


def pack_row(idx, B, row_bytes=None):
    idx = _c(idx, np.int32)
    n = idx.shape[0]
    if row_bytes is None:
        row_bytes = (n * B + 7) // 8
    out = np.empty(row_bytes, np.uint8)
    lib().orc_pack_row(_p(idx), C.c_int(n), C.c_int(B), _p(out), C.c_int64(row_bytes))
    return out


def unpack_row(packed, n_pairs, B):
    packed = _c(packed, np.uint8)
    idx = np.empty(n_pairs, np.int32)
    lib().orc_unpack_row(_p(packed), C.c_int(n_pairs), C.c_int(B), _p(idx))
    return idx


def encode(W, b, codebook, chan_scale, signs, sigma, packed_row_stride=None, diagnostics=False):
    """Full encoder.  Returns a dict with packed [d_out, stride] u8, row_norm f32 and,
    when ``diagnostics``, z f32 [d_out, d_in/2, 2], idx i32, d2_best / d2_second f64."""
    W = np.ascontiguousarray(W)
    d_out, d_in = W.shape
    cb = _c(codebook, np.float32)
    K = cb.shape[0]
    rb = packed_row_bytes(d_in, K)
    stride = rb if packed_row_stride is None else int(packed_row_stride)
    packed = np.zeros((d_out, stride), np.uint8)
    norms = np.empty(d_out, np.float32)
    z = idx = d1 = d2 = None
    if diagnostics:
        z = np.empty((d_out, d_in // 2, 2), np.float32)
        idx = np.empty((d_out, d_in // 2), np.int32)
        d1 = np.empty((d_out, d_in // 2), np.float64)
        d2 = np.empty((d_out, d_in // 2), np.float64)
    rc = lib().orc_encode(_p(W), C.c_int(_w_dtype(W)), C.c_int(d_out), C.c_int(d_in), C.c_int64(d_in),
                          C.c_int(b), C.c_int(K), _p(_c(chan_scale, np.float32)), _p(_c(signs, np.int8)),
                          _p(_c(sigma, np.float32)), _p(cb), _p(packed), C.c_int64(stride), _p(norms),
                          _p(z), _p(idx), _p(d1), _p(d2))
    return dict(status=int(rc), packed=packed, row_norm=norms, z=z, idx=idx, d2_best=d1, d2_second=d2)


def decode(packed, row_norm, b, codebook, chan_scale, signs, sigma, d_in, want_f64=False):
    packed = np.ascontiguousarray(packed, np.uint8)
    d_out, stride = packed.shape
    cb = _c(codebook, np.float32)
    what = np.empty((d_out, d_in), np.uint16)
    w64 = np.empty((d_out, d_in), np.float64) if want_f64 else None
    rc = lib().orc_decode(_p(packed), C.c_int64(stride), _p(_c(row_norm, np.float32)),
                          _p(_c(chan_scale, np.float32)), _p(_c(signs, np.int8)), _p(_c(sigma, np.float32)),
                          _p(cb), C.c_int(cb.shape[0]), C.c_int(b), C.c_int(d_out), C.c_int(d_in),
                          _p(what), _p(w64))
    if rc != ORC_OK:
        raise ValueError(f"orc_decode failed: {rc}")
    return (what, w64) if want_f64 else what


def distortion(W, what_bf16, act_rms=None) -> np.ndarray:
    W = np.ascontiguousarray(W)
    d_out, d_in = W.shape
    wh = np.ascontiguousarray(what_bf16, np.uint16)
    out = np.empty(4, np.float64)
    lib().orc_distortion(_p(W), C.c_int(_w_dtype(W)), C.c_int64(d_in), _p(wh), _p(_c(act_rms, np.float32)),
                         C.c_int(d_out), C.c_int(d_in), _p(out))
    return out


def lloyd_assign(samples, codebook_f64):
    s = _c(samples, np.float64)
    cb = _c(codebook_f64, np.float64)
    assign = np.empty(s.shape[0], np.int32)
    mse = lib().orc_lloyd_assign(_p(s), C.c_uint64(s.shape[0]), _p(cb), C.c_int(cb.shape[0]), _p(assign))
    return assign, float(mse)


def train_codebook(K, n_samples=1 << 20, seed=0, max_iters=100, rel_tol=1e-6, want_trace=False):
    cb = np.empty((K, 2), np.float32)
    mse = C.c_double()
    iters = C.c_int()
    trace = np.full(max_iters + 2, np.nan, np.float64)
    rc = lib().orc_train_codebook(C.c_int(K), C.c_uint64(n_samples), C.c_uint64(seed), C.c_int(max_iters),
                                  C.c_double(rel_tol), _p(cb), C.byref(mse), C.byref(iters), _p(trace))
    if rc != ORC_OK:
        raise ValueError(f"orc_train_codebook failed: {rc}")
    if want_trace:
        return cb, mse.value, iters.value, trace[~np.isnan(trace)]
    return cb, mse.value, iters.value


def train_codebook_on(samples, K, max_iters=100, rel_tol=1e-6):
    """The trainer's iteration on a given [n, 2] float64 sample array -> (codebook f32, mse, updates, trace)."""
    s = _c(samples, np.float64)
    cb = np.empty((K, 2), np.float32)
    mse = C.c_double()
    iters = C.c_int()
    trace = np.full(max_iters + 2, np.nan, np.float64)
    rc = lib().orc_train_codebook_on(_p(s), C.c_uint64(s.shape[0]), C.c_int(K), C.c_int(max_iters), C.c_double(rel_tol),
                                     _p(cb), C.byref(mse), C.byref(iters), _p(trace))
    if rc != ORC_OK:
        raise ValueError(f"orc_train_codebook_on failed: {rc}")
    return cb, mse.value, iters.value, trace[~np.isnan(trace)]


def codebook_mse(codebook, n_samples, seed) -> float:
    cb = _c(codebook, np.float32)
    return float(lib().orc_codebook_mse(_p(cb), C.c_int(cb.shape[0]), C.c_uint64(n_samples), C.c_uint64(seed)))


# ------------------------------------------------------------------------------- polar baseline
def rayleigh_lloyd_max(n_levels: int, max_iters: int = 5000):
    """N-level Lloyd-Max quantiser of the unit Rayleigh density -> (f32 levels, C_LM of those levels)."""
    levels = np.empty(n_levels, np.float32)
    L = lib()
    L.orc_rayleigh_lloyd_max.restype = C.c_double
    c_lm = L.orc_rayleigh_lloyd_max(C.c_int(n_levels), C.c_int(max_iters), _p(levels))
    return levels, float(c_lm)


def rayleigh_distortion(levels) -> float:
    lv = _c(levels, np.float64)
    L = lib()
    L.orc_rayleigh_distortion.restype = C.c_double
    return float(L.orc_rayleigh_distortion(_p(lv), C.c_int(lv.shape[0])))


def polar_codebook(levels, Ba: int, Bp: int) -> np.ndarray:
    lv = _c(levels, np.float32)
    out = np.empty((1 << (Ba + Bp), 2), np.float32)
    lib().orc_polar_codebook(_p(lv), C.c_int(Ba), C.c_int(Bp), _p(out))
    return out


def polar_quantize(z, levels, Ba: int, Bp: int):
    """Polar quantiser for each point of z[n,2] -> (idx, amplitude margin, phase margin)."""
    z = _c(z, np.float64).reshape(-1, 2)
    lv = _c(levels, np.float32)
    idx = np.empty(z.shape[0], np.int32)
    ma = np.empty(z.shape[0], np.float64)
    mp = np.empty(z.shape[0], np.float64)
    L = lib()
    L.orc_polar_quantize.restype = C.c_int
    a, b = C.c_double(), C.c_double()
    for i in range(z.shape[0]):
        idx[i] = L.orc_polar_quantize(C.c_double(z[i, 0]), C.c_double(z[i, 1]), _p(lv), C.c_int(Ba), C.c_int(Bp),
                                      C.byref(a), C.byref(b))
        ma[i], mp[i] = a.value, b.value
    return idx, ma, mp


def encode_polar(W, b, levels, Ba, Bp, chan_scale, signs, sigma, packed_row_stride=None, diagnostics=False):
    """Encoder with the polar quantiser (Section 3.5) instead of the 2-D search."""
    W = np.ascontiguousarray(W)
    d_out, d_in = W.shape
    lv = _c(levels, np.float32)
    K = 1 << (Ba + Bp)
    rb = packed_row_bytes(d_in, K)
    stride = rb if packed_row_stride is None else int(packed_row_stride)
    packed = np.zeros((d_out, stride), np.uint8)
    norms = np.empty(d_out, np.float32)
    z = idx = ma = mp = None
    if diagnostics:
        z = np.empty((d_out, d_in // 2, 2), np.float32)
        idx = np.empty((d_out, d_in // 2), np.int32)
        ma = np.empty((d_out, d_in // 2), np.float64)
        mp = np.empty((d_out, d_in // 2), np.float64)
    rc = lib().orc_encode_polar(_p(W), C.c_int(_w_dtype(W)), C.c_int(d_out), C.c_int(d_in), C.c_int64(d_in),
                                C.c_int(b), C.c_int(Ba), C.c_int(Bp), _p(_c(chan_scale, np.float32)),
                                _p(_c(signs, np.int8)), _p(_c(sigma, np.float32)), _p(lv), _p(packed), C.c_int64(stride),
                                _p(norms), _p(z), _p(idx), _p(ma), _p(mp))
    return dict(status=int(rc), packed=packed, row_norm=norms, z=z, idx=idx, margin_a=ma, margin_p=mp)


# ------------------------------------------------------------------------------- variants
def round_f16(values) -> np.ndarray:
    v = np.array(values, np.float32, copy=True).ravel()
    lib().orc_round_f16(_p(v), C.c_int64(v.shape[0]))
    return v.reshape(np.shape(values))


def renorm_row_norms(packed, row_norm, sigma, codebook, d_in) -> np.ndarray:
    packed = np.ascontiguousarray(packed, np.uint8)
    d_out, stride = packed.shape
    cb = _c(codebook, np.float32)
    out = np.empty(d_out, np.float32)
    rc = lib().orc_renorm_row_norms(_p(packed), C.c_int64(stride), _p(_c(row_norm, np.float32)),
                                    _p(_c(sigma, np.float32)), _p(cb), C.c_int(cb.shape[0]), C.c_int(d_out),
                                    C.c_int(d_in), _p(out))
    if rc != ORC_OK:
        raise ValueError(f"orc_renorm_row_norms failed: {rc}")
    return out
