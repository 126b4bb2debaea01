"""Whole-model driver over the C ABI: calibrate -> encode -> decode -> distortion for every
linear weight of a (synthetic) checkpoint.  This is the call a user of the library makes to
quantise a model.  All four phases go through one qamw_batch: a persistent launch per phase (per
class of row lengths for the encoder side) that walks all matrices.  With ``use_batch = False`` every
phase is one library call per matrix, dealt onto a few side streams.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Optional, Tuple

import numpy as np
import torch

from . import binding as q
from . import synth


def shard_layers(n_layers: int, rank: int, world: int) -> List[int]:
    """Layers owned by `rank` when a model is split over `world` devices: whole layers, round robin.
    Every matrix is independent given its own scales and sigma, so no data crosses devices."""
    if not (0 <= rank < world):
        raise ValueError("rank must be in [0, world)")
    return list(range(rank, n_layers, world))


def combine_distortion(sums4: torch.Tensor, n_weights: int, group=None) -> Dict[str, float]:
    """Model-wide error figures from per-rank sums [sum e^2, sum w^2, sum r^2 e^2, sum r^2 w^2]:
    the only cross-device step of the codec, one all-reduce of five numbers (skipped when
    torch.distributed is not initialised)."""
    import torch.distributed as dist

    v = torch.cat([sums4.detach().to(torch.float64).reshape(4), torch.tensor([float(n_weights)], dtype=torch.float64,
                                                                             device=sums4.device)])
    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(v, op=dist.ReduceOp.SUM, group=group)
    d = v.cpu().numpy()
    return {"rho_w": float(np.sqrt(d[0] / d[1])), "rho_o_diag": float(np.sqrt(d[2] / d[3])),
            "mse": float(d[0] / d[4]), "n_weights": int(d[4])}


def choose_alpha(W: torch.Tensor, act_rms: torch.Tensor, codebook: q.Codebook, block: int,
                 grid=(0.0, 0.3, 0.5, 0.8), sign_seed: int = q.DEFAULT_SIGN_SEED):
    """Scaling exponent for one matrix from the paper's grid {0, 0.3, 0.5, 0.8} (Section B.2 and the
    hyper-parameter table): every candidate goes through channel scales -> calibrate -> encode ->
    decode, and the one with the smallest diagonal-M_x relative output error rho_o (Corollary 4) wins.
    Returns (best alpha, {alpha: (rho_w, rho_o)})."""
    dev = W.device
    d_out, d_in = W.shape
    K = codebook.K
    p = q.make_params(W, d_out, d_in, block, K)
    signs = torch.from_numpy(q.make_signs(sign_seed, d_in)).to(dev)
    sigma = torch.empty(d_in // 2, dtype=torch.float32, device=dev)
    ws = torch.empty(max(8, q.calibrate_workspace_bytes(p)), dtype=torch.uint8, device=dev)
    packed = torch.empty((d_out, p.packed_row_stride), dtype=torch.uint8, device=dev)
    norm = torch.empty(d_out, dtype=torch.float32, device=dev)
    w_hat = torch.empty((d_out, d_in), dtype=torch.bfloat16, device=dev)
    out4 = torch.empty(4, dtype=torch.float64, device=dev)
    act_host = act_rms.detach().cpu().numpy()
    scores = {}
    for alpha in grid:
        s = torch.from_numpy(q.channel_scales(act_host, alpha)).to(dev) if alpha else None
        q.calibrate(W, p, s, signs, sigma, ws)
        q.encode(W, p, s, signs, sigma, codebook, packed, norm)
        q.decode(packed, norm, s, signs, sigma, codebook, p, w_hat)
        q.distortion(W, w_hat, act_rms, p, out4)
        d = out4.cpu().numpy()
        scores[float(alpha)] = (float(np.sqrt(d[0] / d[1])), float(np.sqrt(d[2] / d[3])))
    best = min(scores, key=lambda a: scores[a][1])
    return best, scores


def fit_codebook(W: torch.Tensor, act_rms: Optional[torch.Tensor], alpha: float, block: int, K: int,
                 n_pairs: int = 1 << 20, max_iters: int = 100, rel_tol: float = 1e-6,
                 sign_seed: int = q.DEFAULT_SIGN_SEED, seed: int = 0):
    """Codebook fitted to one matrix's own pairs instead of the unit circular Gaussian (the per-checkpoint
    codebook the paper names as follow-up work, Section 3.6 / Limitations): the rows go through channel
    scaling, normalisation and rotation (qamw_rotate), the pairs are divided by the calibrated pair
    scales, and the device trainer runs Lloyd iterations on up to n_pairs of them (rows taken at a fixed
    stride).  Returns dict(codebook, mse, iters, seconds, sigma, rows)."""
    dev = W.device
    d_out, d_in = W.shape
    p = q.make_params(W, d_out, d_in, block, K)
    signs = torch.from_numpy(q.make_signs(sign_seed, d_in)).to(dev)
    s = None
    if alpha and act_rms is not None:
        s = torch.from_numpy(q.channel_scales(act_rms.detach().cpu().numpy(), alpha)).to(dev)
    sigma = torch.empty(d_in // 2, dtype=torch.float32, device=dev)
    ws = torch.empty(max(8, q.calibrate_workspace_bytes(p)), dtype=torch.uint8, device=dev)
    q.calibrate(W, p, s, signs, sigma, ws)
    n_rows = max(1, min(d_out, (n_pairs + d_in // 2 - 1) // (d_in // 2)))
    rows = torch.div(torch.arange(n_rows, device=dev) * d_out, n_rows, rounding_mode="floor")
    Wsub = W.index_select(0, rows).contiguous()
    ps = q.make_params(Wsub, n_rows, d_in, block, K)
    y = torch.empty((n_rows, d_in), dtype=torch.float32, device=dev)
    norm = torch.empty(n_rows, dtype=torch.float32, device=dev)
    q.rotate(Wsub, ps, s, signs, y, norm)
    z = (y.view(n_rows, d_in // 2, 2) / sigma[None, :, None]).reshape(-1, 2)[:n_pairs].double().contiguous()
    out = q.train_codebook_gpu(K, max_iters=max_iters, rel_tol=rel_tol, samples=z, seed=seed)
    out.update(sigma=sigma, rows=n_rows)
    return out


@dataclass
class MatrixSlot:
    """Device-resident state of one weight matrix."""
    name: str
    d_out: int
    d_in: int
    params: q.Params
    W: torch.Tensor
    act_rms: torch.Tensor
    chan_scale: Optional[torch.Tensor]
    signs: torch.Tensor
    sigma: torch.Tensor
    packed: torch.Tensor
    row_norm: torch.Tensor
    w_hat: torch.Tensor
    dist: torch.Tensor  # 4 doubles


@dataclass
class ModelCodec:
    """All matrices of one workload on one device, plus the shared codebook."""
    spec: synth.WorkloadSpec
    device: torch.device
    codebook: q.Codebook
    slots: List[MatrixSlot] = field(default_factory=list)
    workspace: Optional[torch.Tensor] = None
    status: Optional[torch.Tensor] = None
    batch: Optional[q.Batch] = None
    batch_workspace: Optional[torch.Tensor] = None
    use_batch: bool = True
    _meta_cache: Dict[int, Tuple[torch.Tensor, torch.Tensor]] = field(default_factory=dict)

    @classmethod
    def from_synthetic(cls, spec: synth.WorkloadSpec, device, codebook_host: np.ndarray, rank: int = 0,
                       layers: Optional[List[int]] = None, sign_seed: int = q.DEFAULT_SIGN_SEED) -> "ModelCodec":
        dev = torch.device(device)
        with torch.cuda.device(dev):
            mc = cls(spec, dev, q.Codebook(codebook_host))
            ws_bytes = 8
            for layer, mid, m in synth.iter_matrices(spec, layers):
                seed = synth.matrix_seed(spec, layer, mid, rank)
                W = synth.make_weight(spec, m, seed, device=dev)
                act = synth.make_act_rms(spec, m.d_in, seed, device=dev)
                mc.add_matrix(f"layers.{layer}.{m.name}", W, act, sign_seed)
                ws_bytes = max(ws_bytes, q.calibrate_workspace_bytes(mc.slots[-1].params))
            mc.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
            mc.status = torch.zeros(1, dtype=torch.int32, device=dev)
            mc.finalize()
        return mc

    def finalize(self):
        """Build the batch handle over all matrices added so far (call again after add_matrix)."""
        with torch.cuda.device(self.device):
            mats = [q.make_matrix(s.params, s.W, s.chan_scale, s.signs, s.sigma, s.act_rms, s.packed, s.row_norm,
                                  s.w_hat, s.dist) for s in self.slots]
            self.batch = q.Batch(mats, self.codebook) if mats else None
            self.batch_workspace = (torch.empty(max(8, self.batch.workspace_bytes()), dtype=torch.uint8, device=self.device)
                                    if mats else None)

    def add_matrix(self, name: str, W: torch.Tensor, act_rms: torch.Tensor, sign_seed: int = q.DEFAULT_SIGN_SEED):
        spec, dev = self.spec, self.device
        d_out, d_in = W.shape
        p = q.make_params(W, d_out, d_in, spec.block, spec.K)
        chan_scale = None
        if spec.alpha:
            chan_scale = torch.from_numpy(q.channel_scales(act_rms.cpu().numpy(), spec.alpha)).to(dev)
        if d_in not in self._meta_cache:
            self._meta_cache[d_in] = torch.from_numpy(q.make_signs(sign_seed, d_in)).to(dev)
        self.slots.append(MatrixSlot(
            name, d_out, d_in, p, W, act_rms, chan_scale, self._meta_cache[d_in],
            torch.empty(d_in // 2, dtype=torch.float32, device=dev),
            torch.empty((d_out, p.packed_row_stride), dtype=torch.uint8, device=dev),
            torch.empty(d_out, dtype=torch.float32, device=dev),
            torch.empty((d_out, d_in), dtype=torch.bfloat16, device=dev),
            torch.zeros(4, dtype=torch.float64, device=dev)))

    # --- phases: one library call per matrix ------------------------------------------------------
    # The matrices of a phase are independent, so their launches are dealt round robin onto a few
    # side streams: the next kernel's launch latency and prologue overlap the tail of the previous
    # one.  Every phase forks from and joins back into the caller's current stream, so events
    # recorded there bracket the phase.
    n_streams: int = 4
    _streams: Optional[list] = None
    _workspaces: Optional[list] = None

    def _phase(self, call):
        cur = torch.cuda.current_stream(self.device)
        side_by_side = self.n_streams > 1 and len(self.slots) > 1
        for s in self.slots:  # consecutive matrices then run side by side on half of the SMs each
            s.params.flags = (s.params.flags | q.FLAG_HALF_DEVICE) if side_by_side else (s.params.flags & ~q.FLAG_HALF_DEVICE)
        if not side_by_side:
            for s in self.slots:
                call(s, self.workspace, cur)
            return
        if self._streams is None:
            self._streams = [torch.cuda.Stream(self.device) for _ in range(self.n_streams)]
            self._workspaces = [torch.empty_like(self.workspace) for _ in range(self.n_streams)]
        fork = cur.record_event()
        for st in self._streams:
            st.wait_event(fork)
        for i, s in enumerate(self.slots):
            k = i % self.n_streams
            call(s, self._workspaces[k], self._streams[k])
        for st in self._streams:
            cur.wait_event(st.record_event())

    def calibrate_all(self):
        if self.use_batch and self.batch is not None:
            return self.batch.calibrate(self.batch_workspace, self.status)
        self._phase(lambda s, ws, st: q.calibrate(s.W, s.params, s.chan_scale, s.signs, s.sigma, ws, self.status, st))

    def encode_all(self):
        if self.use_batch and self.batch is not None:
            return self.batch.encode(self.status)
        self._phase(lambda s, ws, st: q.encode(s.W, s.params, s.chan_scale, s.signs, s.sigma, self.codebook, s.packed,
                                               s.row_norm, self.status, st))

    def decode_all(self):
        if self.use_batch and self.batch is not None:
            return self.batch.decode()
        self._phase(lambda s, ws, st: q.decode(s.packed, s.row_norm, s.chan_scale, s.signs, s.sigma, self.codebook,
                                               s.params, s.w_hat, st))

    def distortion_all(self):
        if self.use_batch and self.batch is not None:
            return self.batch.distortion()
        self._phase(lambda s, ws, st: q.distortion(s.W, s.w_hat, s.act_rms, s.params, s.dist, st))

    def step(self):
        """One pass of the whole hot path over the model."""
        self.calibrate_all()
        self.encode_all()
        self.decode_all()
        self.distortion_all()

    def capture_step(self) -> "torch.cuda.CUDAGraph":
        """The whole step as one CUDA graph (seven kernel nodes and a memset for a batched model): replaying
        it costs one launch, which is what small models need -- their kernels take a few microseconds
        each and the per-call overhead of the host dominates otherwise.  The batched phases launch on the
        current stream and allocate nothing, so they can be captured as they are."""
        if not (self.use_batch and self.batch is not None):
            raise RuntimeError("capture_step needs the batched phases (finalize() first)")
        self.step()  # first use outside the capture: per-kernel attributes are set once
        torch.cuda.synchronize(self.device)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.step()
        return graph

    # --- accounting -----------------------------------------------------------------------------
    @property
    def n_weights(self) -> int:
        return sum(s.d_out * s.d_in for s in self.slots)

    def algorithmic_bytes(self) -> Tuple[int, int]:
        """(encode, decode) bytes the codec must move: weights in their dtype, the packed payload
        and 4-byte row norms."""
        enc = dec = 0
        for s in self.slots:
            payload = s.d_out * q.packed_row_bytes(s.d_in, self.spec.K) + 4 * s.d_out
            enc += s.d_out * s.d_in * s.W.element_size() + payload
            dec += s.d_out * s.d_in * 2 + payload
        return enc, dec

    def kernel_launches_per_step(self) -> int:
        # per matrix: calibrate = 2 kernels, distortion 1 (its memset is not a kernel of ours); encode and
        # decode are per matrix too unless batched: then one decode launch and one encode launch per
        # class of row lengths (rows of up to 11264 elements, longer rows)
        n = len(self.slots)
        if self.use_batch and self.batch is not None:
            # one encoder block size per class of row lengths: a calibration pass and an encode launch per
            # class; one finish launch, one decode launch, one distortion launch
            classes = len({self._encoder_class(s.d_in) for s in self.slots})
            return 2 * classes + 3
        return 5 * n

    @staticmethod
    def _encoder_class(d_in: int) -> int:
        n_seg = (d_in + 511) // 512
        best, busy = 0, 0
        for w in (20, 24, 28):
            b = min(15, w // n_seg) * n_seg
            if b > busy:
                best, busy = w, b
        return best

    def totals(self, group=None) -> Dict[str, float]:
        """Error figures over all matrices of all ranks (see combine_distortion)."""
        return combine_distortion(torch.stack([s.dist for s in self.slots]).sum(0), self.n_weights, group)
