"""On-disk form of one encoded weight matrix: everything the decoder needs, in one file.

Layout (little endian): 8 bytes magic, uint32 version, uint32 length of a JSON header, the header,
then the arrays named in the header's "arrays" list, each starting on a 64-byte boundary, in that
order.  The header records shape, block, K, alpha, the sign seed, dtype and shape of every array and
the packed row stride.  With ``f16_metadata`` the row norms, channel scales and sigma are stored as
16-bit floats, which is what the paper's bits-per-weight accounting charges (16 bits per row and per
channel, Section 3.7 / 3.8); they must then already hold f16-representable values (qamw_round_f16),
so that the stored blob decodes to exactly what the in-memory arrays decode to.
"""
from __future__ import annotations

import json
import struct
from typing import Dict, Optional

import numpy as np

MAGIC = b"QAMWBLOB"
VERSION = 1
_ALIGN = 64


def save_blob(path: str, *, d_out: int, d_in: int, block: int, K: int, alpha: float, sign_seed: int,
              codebook: np.ndarray, sigma: np.ndarray, row_norm: np.ndarray, packed: np.ndarray,
              chan_scale: Optional[np.ndarray] = None, f16_metadata: bool = False) -> int:
    """Writes the blob and returns its size in bytes."""
    arrays: Dict[str, np.ndarray] = {"codebook": np.ascontiguousarray(codebook, np.float32),
                                     "packed": np.ascontiguousarray(packed, np.uint8)}
    meta = {"sigma": sigma, "row_norm": row_norm}
    if chan_scale is not None:
        meta["chan_scale"] = chan_scale
    for name, a in meta.items():
        a = np.ascontiguousarray(a, np.float32)
        if f16_metadata:
            h = a.astype(np.float16)
            if not np.array_equal(h.astype(np.float32), a):
                raise ValueError(f"{name} is not f16-representable: round it (qamw_round_f16) before encoding")
            a = h
        arrays[name] = a
    if arrays["packed"].shape[0] != d_out or arrays["codebook"].shape != (K, 2):
        raise ValueError("array shapes do not match the parameters")
    header = {"d_out": d_out, "d_in": d_in, "block": block, "K": K, "alpha": float(alpha), "sign_seed": int(sign_seed),
              "packed_row_stride": int(arrays["packed"].shape[1]),
              "arrays": [{"name": n, "dtype": a.dtype.str, "shape": list(a.shape)} for n, a in arrays.items()]}
    hb = json.dumps(header).encode()
    with open(path, "wb") as f:
        f.write(MAGIC + struct.pack("<II", VERSION, len(hb)) + hb)
        for a in arrays.values():
            f.write(b"\0" * (-f.tell() % _ALIGN))
            f.write(a.tobytes())
        return f.tell()


def load_blob(path: str) -> dict:
    """Reads a blob back: the header fields plus the arrays (metadata widened to float32)."""
    with open(path, "rb") as f:
        raw = f.read()
    if raw[:8] != MAGIC:
        raise ValueError("not a QAM-W blob")
    version, hlen = struct.unpack("<II", raw[8:16])
    if version != VERSION:
        raise ValueError(f"unsupported blob version {version}")
    out = json.loads(raw[16:16 + hlen].decode())
    pos = 16 + hlen
    for spec in out.pop("arrays"):
        pos += -pos % _ALIGN
        dt = np.dtype(spec["dtype"])
        n = int(np.prod(spec["shape"])) * dt.itemsize
        a = np.frombuffer(raw, dt, count=n // dt.itemsize, offset=pos).reshape(spec["shape"]).copy()
        pos += n
        out[spec["name"]] = a.astype(np.float32) if dt == np.float16 else a
    out.setdefault("chan_scale", None)
    return out
