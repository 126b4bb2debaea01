"""Thin ctypes binding of libqamw.so (same names as the C ABI in include/qamw.h).

Only argument marshalling happens here: torch supplies device memory and the
stream, every step of the codec runs inside the library's CUDA kernels.  There
is no fallback: if the shared library is missing or a call fails, an exception
is raised.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass
from typing import Optional, Tuple

import numpy as np
import torch

from . import build as _build

QAMW_OK = 0
ERR_ARG, ERR_SHAPE, ERR_ALIGN, ERR_CUDA, ERR_NONFINITE, ERR_NOMEM = -1, -2, -3, -4, -5, -6
DTYPE_F32, DTYPE_BF16 = 0, 1
FLAG_BRUTE_FORCE = 1
FLAG_HALF_DEVICE = 2
FLAG_GENERAL_KERNELS = 4
DEFAULT_SIGN_SEED = 0x51A5C0DEC0FFEE01
_ERR_NAMES = {-1: "QAMW_ERR_ARG", -2: "QAMW_ERR_SHAPE", -3: "QAMW_ERR_ALIGN", -4: "QAMW_ERR_CUDA",
              -5: "QAMW_ERR_NONFINITE", -6: "QAMW_ERR_NOMEM"}

EXPORTED = [
    "qamw_train_codebook", "qamw_channel_scales", "qamw_make_signs", "qamw_block_size_rule",
    "qamw_packed_row_bytes", "qamw_bpw", "qamw_status_to_error", "qamw_codebook_create",
    "qamw_codebook_destroy", "qamw_codebook_table_info", "qamw_search_table_build",
    "qamw_calibrate_workspace_bytes", "qamw_calibrate", "qamw_calibrate_static", "qamw_encode", "qamw_rotate", "qamw_decode",
    "qamw_distortion", "qamw_last_cuda_error",
    "qamw_batch_create", "qamw_batch_destroy", "qamw_batch_workspace_bytes", "qamw_calibrate_batch",
    "qamw_encode_batch", "qamw_decode_batch", "qamw_distortion_batch",
    "qamw_quantize", "qamw_gemv_workspace_bytes", "qamw_decode_gemv", "qamw_measure_fp32_peak", "qamw_train_codebook_gpu", "qamw_round_f16", "qamw_renorm_row_norms", "qamw_polar_train", "qamw_polar_codebook", "qamw_codebook_create_polar",
]


class QamwError(RuntimeError):
    def __init__(self, fn: str, code: int, detail: str = ""):
        self.code = code
        super().__init__(f"{fn} failed: {_ERR_NAMES.get(code, code)} {detail}".strip())


class Params(C.Structure):
    _fields_ = [("d_out", C.c_int32), ("d_in", C.c_int32), ("block", C.c_int32), ("K", C.c_int32),
                ("w_dtype", C.c_int32), ("flags", C.c_uint32), ("w_row_stride", C.c_int64),
                ("packed_row_stride", C.c_int64)]


class Matrix(C.Structure):
    """qamw_matrix: one weight matrix of a batch (device pointers)."""
    _fields_ = [("p", Params), ("W", C.c_void_p), ("chan_scale", C.c_void_p), ("signs", C.c_void_p),
                ("sigma", C.c_void_p), ("act_rms", C.c_void_p), ("packed", C.c_void_p), ("row_norm", C.c_void_p),
                ("w_hat_bf16", C.c_void_p), ("dist4", C.c_void_p)]


_lib = None


def lib() -> C.CDLL:
    """Loads libqamw.so from the package directory; raises if it has not been built."""
    global _lib
    if _lib is None:
        path = _build.LIB_PATH
        if not os.path.exists(path):
            raise RuntimeError(f"{path} is missing: run __graft_entry__.build() (nvcc, sm_100a) first; "
                               "there is no CPU fallback")
        L = C.CDLL(path)
        vp, i32, u64, sz = C.c_void_p, C.c_int, C.c_uint64, C.c_size_t
        L.qamw_train_codebook.argtypes = [i32, u64, u64, i32, C.c_double, vp, vp]
        L.qamw_channel_scales.argtypes = [vp, i32, C.c_float, vp]
        L.qamw_make_signs.argtypes = [u64, i32, vp]
        L.qamw_block_size_rule.argtypes = [i32]
        L.qamw_packed_row_bytes.argtypes = [i32, i32]
        L.qamw_packed_row_bytes.restype = sz
        L.qamw_bpw.argtypes = [i32, i32, i32, i32]
        L.qamw_bpw.restype = C.c_double
        L.qamw_status_to_error.argtypes = [C.c_int32]
        L.qamw_codebook_create.argtypes = [vp, i32, i32, C.POINTER(vp)]
        L.qamw_codebook_destroy.argtypes = [vp]
        L.qamw_codebook_destroy.restype = None
        L.qamw_codebook_table_info.argtypes = [vp, vp]
        L.qamw_search_table_build.argtypes = [vp, i32, i32, sz, vp, vp, sz, vp, sz, vp]
        L.qamw_calibrate_workspace_bytes.argtypes = [C.POINTER(Params)]
        L.qamw_calibrate_workspace_bytes.restype = sz
        L.qamw_calibrate.argtypes = [vp, C.POINTER(Params), vp, vp, vp, vp, sz, vp, vp]
        L.qamw_calibrate_static.argtypes = [vp, C.POINTER(Params), vp, vp, vp, vp, vp]
        L.qamw_encode.argtypes = [vp, C.POINTER(Params), vp, vp, vp, vp, vp, vp, vp, vp]
        L.qamw_rotate.argtypes = [vp, C.POINTER(Params), vp, vp, vp, vp, vp, vp]
        L.qamw_decode.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Params), vp, vp]
        L.qamw_distortion.argtypes = [vp, vp, vp, C.POINTER(Params), vp, vp]
        L.qamw_last_cuda_error.restype = C.c_char_p
        L.qamw_train_codebook_gpu.argtypes = [i32, u64, u64, vp, i32, C.c_double, vp, vp, vp, vp, vp]
        L.qamw_quantize.argtypes = [vp, C.POINTER(Params), vp, C.c_float, u64, vp, vp, vp, vp, vp, vp, vp, sz, vp, vp]
        L.qamw_gemv_workspace_bytes.argtypes = [C.POINTER(Params), i32]
        L.qamw_gemv_workspace_bytes.restype = sz
        L.qamw_decode_gemv.argtypes = [vp, vp, vp, vp, vp, vp, C.POINTER(Params), vp, i32, vp, vp, sz, vp]
        L.qamw_measure_fp32_peak.argtypes = [vp, vp]
        L.qamw_round_f16.argtypes = [vp, sz, vp]
        L.qamw_renorm_row_norms.argtypes = [vp, vp, vp, vp, C.POINTER(Params), vp, vp]
        L.qamw_polar_train.argtypes = [i32, vp, vp]
        L.qamw_polar_codebook.argtypes = [vp, i32, i32, vp]
        L.qamw_codebook_create_polar.argtypes = [vp, i32, i32, C.POINTER(vp)]
        L.qamw_batch_create.argtypes = [C.POINTER(Matrix), i32, vp, C.POINTER(vp)]
        L.qamw_batch_destroy.argtypes = [vp]
        L.qamw_batch_destroy.restype = None
        L.qamw_batch_workspace_bytes.argtypes = [vp]
        L.qamw_batch_workspace_bytes.restype = sz
        L.qamw_calibrate_batch.argtypes = [vp, vp, sz, vp, vp]
        L.qamw_encode_batch.argtypes = [vp, vp, vp]
        L.qamw_decode_batch.argtypes = [vp, vp]
        L.qamw_distortion_batch.argtypes = [vp, vp]
        _lib = L
    return _lib


def _check(fn: str, rc: int):
    if rc != QAMW_OK:
        detail = lib().qamw_last_cuda_error().decode() if rc == ERR_CUDA else ""
        raise QamwError(fn, rc, detail)


def _np(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def _dp(t: Optional[torch.Tensor]):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


# ------------------------------------------------------------------------------- host side
def train_codebook(K: int, n_samples: int = 1 << 20, seed: int = 0, max_iters: int = 100,
                   rel_tol: float = 1e-6) -> Tuple[np.ndarray, float]:
    cb = np.empty((K, 2), np.float32)
    mse = C.c_double()
    _check("qamw_train_codebook", lib().qamw_train_codebook(K, n_samples, seed, max_iters, rel_tol,
                                                           cb.ctypes.data, C.addressof(mse)))
    return cb, mse.value


def train_codebook_gpu(K: int, n_samples: int = 1 << 20, seed: int = 0, max_iters: int = 100, rel_tol: float = 1e-6,
                       samples: Optional[torch.Tensor] = None):
    """Lloyd training on the current CUDA device -> dict(codebook, mse, iters, trace, seconds).
    samples: optional float64 device tensor [n, 2] to train on instead of the generated Gaussian."""
    cb = np.empty((K, 2), np.float32)
    mse, secs, iters = C.c_double(), C.c_double(), C.c_int()
    trace = np.full(max_iters + 2, np.nan, np.float64)
    if samples is not None:
        if samples.dtype != torch.float64 or samples.dim() != 2 or samples.shape[1] != 2 or not samples.is_contiguous():
            raise TypeError("samples must be a contiguous float64 [n, 2] device tensor")
        n_samples = samples.shape[0]
    _check("qamw_train_codebook_gpu", lib().qamw_train_codebook_gpu(
        K, n_samples, seed, _dp(samples), max_iters, rel_tol, cb.ctypes.data, C.addressof(mse), C.addressof(iters),
        trace.ctypes.data, C.addressof(secs)))
    return dict(codebook=cb, mse=mse.value, iters=iters.value, trace=trace[~np.isnan(trace)], seconds=secs.value)


def channel_scales(act_rms, alpha: float) -> np.ndarray:
    r = _np(act_rms, np.float32)
    out = np.empty_like(r)
    _check("qamw_channel_scales", lib().qamw_channel_scales(r.ctypes.data, r.shape[0], alpha, out.ctypes.data))
    return out


def make_signs(seed: int, d_in: int) -> np.ndarray:
    out = np.empty(d_in, np.int8)
    _check("qamw_make_signs", lib().qamw_make_signs(seed, d_in, out.ctypes.data))
    return out


def block_size_rule(d_in: int) -> int:
    return int(lib().qamw_block_size_rule(d_in))


def packed_row_bytes(d_in: int, K: int) -> int:
    return int(lib().qamw_packed_row_bytes(d_in, K))


def bpw(d_out: int, d_in: int, K: int, has_channel_scales: bool) -> float:
    return float(lib().qamw_bpw(d_out, d_in, K, int(has_channel_scales)))


def status_to_error(status_word: int) -> int:
    return int(lib().qamw_status_to_error(status_word))


def polar_train(Ba: int) -> Tuple[np.ndarray, float]:
    """Lloyd-Max amplitude levels of the polar baseline -> (f32 levels[2^Ba], C_LM)."""
    lv = np.empty(1 << Ba, np.float32)
    c = C.c_double()
    _check("qamw_polar_train", lib().qamw_polar_train(Ba, lv.ctypes.data, C.addressof(c)))
    return lv, c.value


def polar_codebook(levels, Ba: int, Bp: int) -> np.ndarray:
    lv = _np(levels, np.float32)
    out = np.empty((1 << (Ba + Bp), 2), np.float32)
    _check("qamw_polar_codebook", lib().qamw_polar_codebook(lv.ctypes.data, Ba, Bp, out.ctypes.data))
    return out


def search_table_build(codebook, grid: int = 0, budget_bytes: int = 1 << 20):
    """Host-only table construction -> (map f32[4] = zmax, c0, c1, c2; cells u16[grid*grid,4]; overflow u16[];
    info[6])."""
    cb = _np(codebook, np.float32)
    K = cb.shape[0]
    info = np.zeros(6, np.int32)
    _check("qamw_search_table_build", lib().qamw_search_table_build(cb.ctypes.data, K, grid, budget_bytes, None,
                                                                    None, 0, None, 0, info.ctypes.data))
    g = int(info[0])
    cmap = np.zeros(4, np.float32)
    cells = np.zeros((g * g, 4), np.uint16)
    ovf = np.zeros(max(1, int(info[4])), np.uint16)
    _check("qamw_search_table_build", lib().qamw_search_table_build(cb.ctypes.data, K, g, budget_bytes,
                                                                    cmap.ctypes.data, cells.ctypes.data, cells.size,
                                                                    ovf.ctypes.data, ovf.size, info.ctypes.data))
    return cmap, cells, ovf, info


# ------------------------------------------------------------------------------- codebook object
class Codebook:
    """Owns a qamw_codebook* on the current CUDA device."""

    def __init__(self, codebook, grid: int = 0):
        cb = _np(codebook, np.float32)
        if cb.ndim != 2 or cb.shape[1] != 2:
            raise ValueError("codebook must be [K, 2]")
        self.K = cb.shape[0]
        self.host = cb.copy()
        h = C.c_void_p()
        _check("qamw_codebook_create", lib().qamw_codebook_create(cb.ctypes.data, self.K, grid, C.byref(h)))
        self._h = h

    @classmethod
    def polar(cls, levels, Ba: int, Bp: int) -> "Codebook":
        """Codebook object of the polar baseline quantiser (qamw_codebook_create_polar)."""
        lv = _np(levels, np.float32)
        self = cls.__new__(cls)
        self.K = 1 << (Ba + Bp)
        self.host = polar_codebook(lv, Ba, Bp)
        h = C.c_void_p()
        _check("qamw_codebook_create_polar", lib().qamw_codebook_create_polar(lv.ctypes.data, Ba, Bp, C.byref(h)))
        self._h = h
        return self

    @property
    def handle(self):
        return self._h

    def table_info(self) -> np.ndarray:
        info = np.zeros(6, np.int32)
        _check("qamw_codebook_table_info", lib().qamw_codebook_table_info(self._h, info.ctypes.data))
        return info

    def close(self):
        if getattr(self, "_h", None):
            lib().qamw_codebook_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


# ------------------------------------------------------------------------------- device side
@dataclass
class MatrixMeta:
    """Device-resident per-matrix metadata shared by encode and decode."""
    chan_scale: Optional[torch.Tensor]  # f32 [d_in] or None
    signs: torch.Tensor  # int8 [d_in]
    sigma: Optional[torch.Tensor]  # f32 [d_in/2]


def make_params(W: Optional[torch.Tensor], d_out: int, d_in: int, block: int, K: int, flags: int = 0,
                packed_row_stride: Optional[int] = None, w_dtype: Optional[int] = None) -> Params:
    if W is not None:
        if W.dtype == torch.float32:
            w_dtype = DTYPE_F32
        elif W.dtype == torch.bfloat16:
            w_dtype = DTYPE_BF16
        else:
            raise TypeError("W must be float32 or bfloat16")
        if W.dim() != 2 or W.stride(1) != 1:
            raise ValueError("W must be 2-D with unit column stride")
        stride = W.stride(0) if W.shape[0] > 1 else d_in
    else:
        stride = d_in
        w_dtype = DTYPE_BF16 if w_dtype is None else w_dtype
    if packed_row_stride is None:
        packed_row_stride = default_packed_row_stride(d_in, K)
    return Params(d_out, d_in, block, K, w_dtype, flags, stride, packed_row_stride)


def default_packed_row_stride(d_in: int, K: int) -> int:
    """Row payload rounded up to 4 bytes (16 when the payload already is a multiple of 16)."""
    rb = packed_row_bytes(d_in, K)
    return (rb + 3) // 4 * 4


def calibrate_workspace_bytes(p: Params) -> int:
    return int(lib().qamw_calibrate_workspace_bytes(C.byref(p)))


def calibrate(W: torch.Tensor, p: Params, chan_scale, signs, sigma_out: torch.Tensor, workspace: torch.Tensor,
              status: Optional[torch.Tensor] = None, stream=None):
    _check("qamw_calibrate", lib().qamw_calibrate(_dp(W), C.byref(p), _dp(chan_scale), _dp(signs), _dp(sigma_out),
                                                 _dp(workspace), workspace.numel() * workspace.element_size(),
                                                 _dp(status), _stream(stream)))


STATIC_SCRATCH_BYTES = 16 << 20


def calibrate_static(W: torch.Tensor, p: Params, chan_scale, signs, sigma_out: torch.Tensor,
                     status: Optional[torch.Tensor] = None, stream=None):
    """qamw_calibrate without a caller-provided workspace: for hosts that may not allocate device
    memory.  The partial sums live in a 16 MiB array built into the library; calls on one device
    share it, so calls that could overlap on the GPU must be ordered by the caller."""
    rc = lib().qamw_calibrate_static(_dp(W), C.byref(p), _dp(chan_scale), _dp(signs), _dp(sigma_out), _dp(status),
                                     _stream(stream))
    if rc == ERR_NOMEM:
        raise QamwError("qamw_calibrate_static", rc, lib().qamw_last_cuda_error().decode())
    _check("qamw_calibrate_static", rc)


def encode(W: torch.Tensor, p: Params, chan_scale, signs, sigma, cb: Codebook, packed_out: torch.Tensor,
           row_norm_out: torch.Tensor, status: Optional[torch.Tensor] = None, stream=None):
    _check("qamw_encode", lib().qamw_encode(_dp(W), C.byref(p), _dp(chan_scale), _dp(signs), _dp(sigma), cb.handle,
                                           _dp(packed_out), _dp(row_norm_out), _dp(status), _stream(stream)))


def quantize(W: torch.Tensor, p: Params, act_rms, alpha: float, sign_seed: int, cb: Codebook, chan_scale_out,
             signs_out: torch.Tensor, sigma_out: torch.Tensor, packed_out: torch.Tensor, row_norm_out: torch.Tensor,
             workspace: torch.Tensor, status: Optional[torch.Tensor] = None, stream=None):
    """qamw_quantize: channel scales -> signs -> calibrate -> encode in one call (act_rms: host array or None)."""
    r = None if act_rms is None else _np(act_rms, np.float32)
    _check("qamw_quantize", lib().qamw_quantize(
        _dp(W), C.byref(p), None if r is None else r.ctypes.data, alpha, sign_seed, cb.handle, _dp(chan_scale_out),
        _dp(signs_out), _dp(sigma_out), _dp(packed_out), _dp(row_norm_out), _dp(workspace),
        workspace.numel() * workspace.element_size(), _dp(status), _stream(stream)))


def rotate(W: torch.Tensor, p: Params, chan_scale, signs, y_out: torch.Tensor, row_norm_out: torch.Tensor,
           status: Optional[torch.Tensor] = None, stream=None):
    _check("qamw_rotate", lib().qamw_rotate(_dp(W), C.byref(p), _dp(chan_scale), _dp(signs), _dp(y_out),
                                           _dp(row_norm_out), _dp(status), _stream(stream)))


def decode(packed: torch.Tensor, row_norm: torch.Tensor, chan_scale, signs, sigma, cb: Codebook, p: Params,
           w_hat_out: torch.Tensor, stream=None):
    _check("qamw_decode", lib().qamw_decode(_dp(packed), _dp(row_norm), _dp(chan_scale), _dp(signs), _dp(sigma),
                                           cb.handle, C.byref(p), _dp(w_hat_out), _stream(stream)))


def decode_gemv(packed: torch.Tensor, row_norm: torch.Tensor, chan_scale, signs, sigma, cb: Codebook, p: Params,
                x: torch.Tensor, y_out: torch.Tensor, workspace: Optional[torch.Tensor] = None, stream=None):
    """y = W_hat x straight from the packed stream (x: float32 [n_vec, d_in], y_out: float32 [d_out, n_vec])."""
    n_vec = x.shape[0]
    if workspace is None:
        workspace = torch.empty(int(lib().qamw_gemv_workspace_bytes(C.byref(p), n_vec)), dtype=torch.uint8, device=x.device)
    _check("qamw_decode_gemv", lib().qamw_decode_gemv(
        _dp(packed), _dp(row_norm), _dp(chan_scale), _dp(signs), _dp(sigma), cb.handle, C.byref(p), _dp(x), n_vec,
        _dp(y_out), _dp(workspace), workspace.numel(), _stream(stream)))


def measure_fp32_peak() -> float:
    """Plain FP32 lane instructions per second of the current device (FMA micro-benchmark)."""
    scratch = torch.zeros(1, dtype=torch.float32, device="cuda")
    out = C.c_double()
    _check("qamw_measure_fp32_peak", lib().qamw_measure_fp32_peak(_dp(scratch), C.addressof(out)))
    return out.value


def round_f16(values: torch.Tensor, stream=None):
    """Rounds a float32 device tensor in place to what a 16-bit (f16) serialisation would hold."""
    if values.dtype != torch.float32 or not values.is_contiguous():
        raise TypeError("values must be a contiguous float32 tensor")
    _check("qamw_round_f16", lib().qamw_round_f16(_dp(values), values.numel(), _stream(stream)))


def renorm_row_norms(packed: torch.Tensor, row_norm: torch.Tensor, sigma, cb: Codebook, p: Params,
                     row_norm_out: torch.Tensor, stream=None):
    _check("qamw_renorm_row_norms", lib().qamw_renorm_row_norms(_dp(packed), _dp(row_norm), _dp(sigma), cb.handle,
                                                               C.byref(p), _dp(row_norm_out), _stream(stream)))


def distortion(W: torch.Tensor, w_hat: torch.Tensor, act_rms, p: Params, out4: torch.Tensor, stream=None):
    _check("qamw_distortion", lib().qamw_distortion(_dp(W), _dp(w_hat), _dp(act_rms), C.byref(p), _dp(out4),
                                                   _stream(stream)))


# ------------------------------------------------------------------------------- batches
def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def make_matrix(p: Params, W=None, chan_scale=None, signs=None, sigma=None, act_rms=None, packed=None,
                row_norm=None, w_hat=None, dist4=None) -> Matrix:
    """qamw_matrix from torch tensors (device); the caller keeps the tensors alive."""
    return Matrix(p, _ptr(W), _ptr(chan_scale), _ptr(signs), _ptr(sigma), _ptr(act_rms), _ptr(packed),
                  _ptr(row_norm), _ptr(w_hat), _ptr(dist4))


class Batch:
    """Owns a qamw_batch* (all matrices of a layer or model) on the current CUDA device."""

    def __init__(self, matrices, cb: Codebook):
        self.n = len(matrices)
        arr = (Matrix * self.n)(*matrices)
        self._cb = cb  # the codebook must outlive the batch
        h = C.c_void_p()
        _check("qamw_batch_create", lib().qamw_batch_create(arr, self.n, cb.handle, C.byref(h)))
        self._h = h

    def workspace_bytes(self) -> int:
        return int(lib().qamw_batch_workspace_bytes(self._h))

    def calibrate(self, workspace: torch.Tensor, status: Optional[torch.Tensor] = None, stream=None):
        _check("qamw_calibrate_batch", lib().qamw_calibrate_batch(
            self._h, _dp(workspace), workspace.numel() * workspace.element_size(), _dp(status), _stream(stream)))

    def encode(self, status: Optional[torch.Tensor] = None, stream=None):
        _check("qamw_encode_batch", lib().qamw_encode_batch(self._h, _dp(status), _stream(stream)))

    def decode(self, stream=None):
        _check("qamw_decode_batch", lib().qamw_decode_batch(self._h, _stream(stream)))

    def distortion(self, stream=None):
        _check("qamw_distortion_batch", lib().qamw_distortion_batch(self._h, _stream(stream)))

    def close(self):
        if getattr(self, "_h", None):
            lib().qamw_batch_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
