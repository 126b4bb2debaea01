"""The on-disk blob of one encoded matrix: round trip, alignment, and the file's bits per weight
against the closed form of Section 3.7 (B/2 + 16/d_in, plus 16/d_out with channel scales)."""
import os

import numpy as np
import pytest

from paper_2605_26339_b200 import blob


def _arrays(orc, d_out, d_in, K, f16):
    rng = np.random.default_rng(2)
    B = int(np.log2(K))
    idx = rng.integers(0, K, (d_out, d_in // 2))
    packed = np.stack([orc.pack_row(r, B) for r in idx])
    meta = [np.exp(rng.standard_normal(n)).astype(np.float32) for n in (d_in // 2, d_out, d_in)]
    if f16:
        meta = [orc.round_f16(m) for m in meta]
    cb = rng.standard_normal((K, 2)).astype(np.float32)
    return cb, packed, meta


@pytest.mark.parametrize("f16", [False, True])
def test_blob_round_trip(orc, tmp_path, f16):
    d_out, d_in, K = 24, 4096, 2048
    cb, packed, (sigma, norm, s) = _arrays(orc, d_out, d_in, K, f16)
    path = os.path.join(tmp_path, "m.qamw")
    size = blob.save_blob(path, d_out=d_out, d_in=d_in, block=128, K=K, alpha=0.3, sign_seed=7, codebook=cb, sigma=sigma,
                          row_norm=norm, packed=packed, chan_scale=s, f16_metadata=f16)
    assert size == os.path.getsize(path)
    b = blob.load_blob(path)
    assert (b["d_out"], b["d_in"], b["block"], b["K"], b["sign_seed"]) == (d_out, d_in, 128, K, 7)
    assert np.array_equal(b["packed"], packed) and np.array_equal(b["codebook"], cb)
    assert np.array_equal(b["sigma"], sigma) and np.array_equal(b["row_norm"], norm) and np.array_equal(b["chan_scale"], s)
    if f16:
        # payload + 16 bits per row and per channel; what is left is the shared part: codebook, sigma
        # (2 bytes per pair position, shared by all rows), header and alignment padding
        per_matrix = d_out * d_in * orc.bpw(d_out, d_in, K, True) / 8
        assert 0 <= size - per_matrix - cb.nbytes - sigma.size * 2 < 1024


def test_blob_refuses_unrounded_metadata_and_foreign_files(orc, tmp_path):
    cb, packed, (sigma, norm, s) = _arrays(orc, 4, 256, 16, False)
    with pytest.raises(ValueError):
        blob.save_blob(os.path.join(tmp_path, "x"), d_out=4, d_in=256, block=64, K=16, alpha=0, sign_seed=1, codebook=cb,
                       sigma=sigma, row_norm=norm, packed=packed, f16_metadata=True)
    bad = os.path.join(tmp_path, "bad")
    open(bad, "wb").write(b"nonsense" * 8)
    with pytest.raises(ValueError):
        blob.load_blob(bad)
