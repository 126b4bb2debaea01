import os
import sys

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)
GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run on a B200 with -m gpu)")


def load_golden_codebook(K: int) -> np.ndarray:
    """Oracle-trained codebook written by tests/golden/make_codebooks.py."""
    rows = []
    with open(os.path.join(GOLDEN, f"codebook_K{K}.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            a, b = line.split()
            rows.append((int(a, 16), int(b, 16)))
    cb = np.array(rows, dtype=np.uint32).view(np.float32)
    assert cb.shape == (K, 2)
    return cb


def golden_header(K: int) -> dict:
    out = {}
    with open(os.path.join(GOLDEN, f"codebook_K{K}.txt")) as f:
        for line in f:
            if not line.startswith("#"):
                break
            for tok in line[1:].split():
                if "=" in tok:
                    k, v = tok.split("=", 1)
                    out[k] = v.rstrip(",")
    return out


@pytest.fixture(scope="session")
def orc():
    from oracle import oracle
    oracle.build()
    return oracle
