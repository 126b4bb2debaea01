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
    # the shared library is built in-tree (nvcc cross-compiles without a GPU); a box without nvcc
    # uses the copy that travelled with the repository
    import shutil
    from paper_2605_26339_b200 import build as lib_build
    if lib_build.needs_build() and (shutil.which("nvcc") or os.path.exists("/usr/local/cuda/bin/nvcc")):
        lib_build.build()


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
