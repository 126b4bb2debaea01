"""Seeded synthetic inputs shaped like the paper's workloads.

This module holds no codec arithmetic: it only draws weight matrices and
activation statistics with the shapes and value distributions of the benchmark
configurations, so that the CUDA library and the test oracle can be fed the very
same bits.  The paper quantises real checkpoints (TinyLlama-1.1B ... Llama-2-13B,
Section 5 and Appendix F); those are not available offline, so tensors with the
public architecture shapes and heavy-tailed entries stand in for them.

Everything is drawn with ``torch`` generators (CPU or CUDA).  A CPU and a CUDA
generator with the same seed give different streams; parity tests always copy
the generated bits to the other side instead of regenerating them.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional, Tuple

import torch


@dataclass(frozen=True)
class MatrixSpec:
    name: str
    d_out: int
    d_in: int


@dataclass(frozen=True)
class WorkloadSpec:
    """One benchmark configuration: which matrices, how they are drawn, codec parameters."""
    name: str
    matrices: Tuple[MatrixSpec, ...]  # matrices of ONE layer
    n_layers: int
    w_dtype: str  # "f32" | "bf16"
    entry: str  # "normal" | "student_t"
    nu: int  # degrees of freedom for student_t
    row_sigma: float  # lognormal(0, row_sigma) per-row scale
    col_outlier_frac: float  # fraction of weight columns multiplied by col_outlier_gain
    col_outlier_gain: float
    act_outlier_frac: float  # fraction of activation channels multiplied by act_outlier_gain
    act_outlier_gain: float
    alpha: float
    block: int
    K: int
    base_seed: int

    @property
    def n_weights(self) -> int:
        return self.n_layers * sum(m.d_out * m.d_in for m in self.matrices)

    @property
    def n_rows(self) -> int:
        return self.n_layers * sum(m.d_out for m in self.matrices)


def decoder_layer(hidden: int, inter: int, kv_dim: Optional[int] = None) -> Tuple[MatrixSpec, ...]:
    kv = hidden if kv_dim is None else kv_dim
    return (
        MatrixSpec("q_proj", hidden, hidden),
        MatrixSpec("k_proj", kv, hidden),
        MatrixSpec("v_proj", kv, hidden),
        MatrixSpec("o_proj", hidden, hidden),
        MatrixSpec("gate_proj", inter, hidden),
        MatrixSpec("up_proj", inter, hidden),
        MatrixSpec("down_proj", hidden, inter),
    )


def workload(name: str, K: Optional[int] = None, block: Optional[int] = None) -> WorkloadSpec:
    """The five benchmark configurations ("cfg0" .. "cfg4")."""
    if name == "cfg0":  # single FP32 layer, Gaussian entries
        w = WorkloadSpec("cfg0", (MatrixSpec("linear", 1024, 1024),), 1, "f32", "normal", 0, 0.5,
                         0.0, 1.0, 0.01, 20.0, 0.5, 128, 256, 1000)
    elif name == "cfg1":  # one 7B-style decoder layer
        w = WorkloadSpec("cfg1", decoder_layer(4096, 11008), 1, "bf16", "student_t", 5, 0.5,
                         0.005, 10.0, 0.01, 20.0, 0.3, 128, 2048, 1001)
    elif name == "cfg2":  # TinyLlama-1.1B shape
        w = WorkloadSpec("cfg2", decoder_layer(2048, 5632, 256), 22, "bf16", "normal", 0, 0.5,
                         0.0, 1.0, 0.0, 1.0, 0.3, 128, 2048, 1002)
    elif name == "cfg3":  # Llama-2-13B shape
        w = WorkloadSpec("cfg3", decoder_layer(5120, 13824), 40, "bf16", "student_t", 4, 0.7,
                         0.01, 20.0, 0.01, 20.0, 0.3, 128, 2048, 1003)
    elif name == "cfg4":  # sweep matrix
        w = WorkloadSpec("cfg4", (MatrixSpec("gate_proj", 13824, 5120),), 1, "bf16", "student_t", 4, 0.7,
                         0.01, 20.0, 0.01, 20.0, 0.3, 128, 2048, 1004)
    else:
        raise KeyError(name)
    if K is not None or block is not None:
        w = WorkloadSpec(**{**w.__dict__, "K": K or w.K, "block": block or w.block})
    return w


def matrix_seed(spec: WorkloadSpec, layer: int, matrix_id: int, rank: int = 0) -> int:
    return spec.base_seed + 16 * layer + matrix_id + 1_000_003 * rank


def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def make_weight(spec: WorkloadSpec, m: MatrixSpec, seed: int, device="cpu", row_chunk: int = 2048) -> torch.Tensor:
    """Draw one weight matrix [d_out, d_in] in the workload's dtype (f32 or bf16)."""
    dev = torch.device(device)
    g = _gen(dev, seed)
    out_dtype = torch.float32 if spec.w_dtype == "f32" else torch.bfloat16
    W = torch.empty((m.d_out, m.d_in), dtype=out_dtype, device=dev)
    col_gain = torch.ones(m.d_in, dtype=torch.float32, device=dev)
    if spec.col_outlier_frac > 0:
        n_out = max(1, int(round(spec.col_outlier_frac * m.d_in)))
        cols = torch.randperm(m.d_in, generator=g, device=dev)[:n_out]
        col_gain[cols] = spec.col_outlier_gain
    for r0 in range(0, m.d_out, row_chunk):
        r1 = min(m.d_out, r0 + row_chunk)
        n = r1 - r0
        x = torch.randn((n, m.d_in), generator=g, device=dev, dtype=torch.float32)
        if spec.entry == "student_t":
            chi = torch.zeros_like(x)
            for _ in range(spec.nu):
                chi += torch.randn((n, m.d_in), generator=g, device=dev, dtype=torch.float32) ** 2
            x = x / torch.sqrt(chi / spec.nu)
        row_scale = torch.exp(spec.row_sigma * torch.randn((n, 1), generator=g, device=dev, dtype=torch.float32))
        W[r0:r1] = (x * row_scale * col_gain).to(out_dtype)
    return W


def make_act_rms(spec: WorkloadSpec, d_in: int, seed: int, device="cpu") -> torch.Tensor:
    """Per-input-channel activation RMS: lognormal(0,1) with a few amplified channels."""
    dev = torch.device(device)
    g = _gen(dev, seed ^ 0x5EED)
    r = torch.exp(torch.randn(d_in, generator=g, device=dev, dtype=torch.float32))
    if spec.act_outlier_frac > 0:
        n_out = max(1, int(round(spec.act_outlier_frac * d_in)))
        ch = torch.randperm(d_in, generator=g, device=dev)[:n_out]
        r[ch] *= spec.act_outlier_gain
    return r


def iter_matrices(spec: WorkloadSpec, layers: Optional[List[int]] = None):
    """Yield (layer, matrix_id, MatrixSpec) for the whole workload."""
    for layer in (range(spec.n_layers) if layers is None else layers):
        for mid, m in enumerate(spec.matrices):
            yield layer, mid, m


def algorithmic_bytes_per_weight(spec: WorkloadSpec, d_in: int) -> Tuple[float, float]:
    """(encode, decode) bytes the codec must move per weight: the weight itself
    (input dtype for encode, bf16 for decode), B/16 bytes of packed index and a
    4-byte row norm per d_in weights."""
    B = int(math.log2(spec.K))
    w_in = 4.0 if spec.w_dtype == "f32" else 2.0
    return w_in + B / 16.0 + 4.0 / d_in, 2.0 + B / 16.0 + 4.0 / d_in
