"""Writes tests/golden/codebook_K*.txt by calling ONLY the CPU oracle.

Each file is the 2-D Lloyd-Max codebook the oracle trains on 2^20 unit
circular-Gaussian samples, seed 0, at most 100 centroid updates, relative
stopping tolerance 1e-6 (Section 3.6 of the paper describes the training as
"Lloyd iterations on the unit circular Gaussian"; sample count, seed,
initialisation and stopping rule are this repository's reading).  One codeword
per line as two IEEE-754 binary32 bit patterns in hex, in index order; header
lines start with '#'.

Run from the repository root:  python tests/golden/make_codebooks.py [K ...]
"""
import os
import sys
import time

import numpy as np

sys.path.insert(0, os.path.join(os.path.dirname(os.path.abspath(__file__)), "..", ".."))
from oracle import oracle as orc  # noqa: E402

N_SAMPLES = 1 << 20
SEED = 0
MAX_ITERS = 100
REL_TOL = 1e-6


def main(argv):
    ks = [int(a) for a in argv] or [64, 128, 256, 1024, 2048, 4096]
    here = os.path.dirname(os.path.abspath(__file__))
    for K in ks:
        t0 = time.time()
        cb, mse, iters = orc.train_codebook(K, N_SAMPLES, SEED, MAX_ITERS, REL_TOL)
        path = os.path.join(here, f"codebook_K{K}.txt")
        with open(path, "w") as f:
            f.write(f"# 2-D Lloyd-Max codebook, K={K}, oracle-trained (Section 3.6)\n")
            f.write(f"# n_samples={N_SAMPLES} seed={SEED} max_iters={MAX_ITERS} rel_tol={REL_TOL}\n")
            f.write(f"# centroid_updates={iters} train_mse={mse:.12e}\n")
            bits = np.ascontiguousarray(cb, np.float32).view(np.uint32)
            for c in range(K):
                f.write(f"{bits[c, 0]:08x} {bits[c, 1]:08x}\n")
        print(f"K={K}: updates={iters} mse={mse:.6e} ({time.time() - t0:.1f}s) -> {path}", flush=True)


if __name__ == "__main__":
    main(sys.argv[1:])
