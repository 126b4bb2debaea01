"""Two CPU processes over gloo stand in for two GPUs: each takes the layers that shard_layers gives
it, runs the codec on them (here with the oracle, since there is no GPU), and the model-wide error
figures come from combine_distortion's single all-reduce.  They must equal what one process computes
over the whole model."""
import os
import sys

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from conftest import ROOT, load_golden_codebook

TINY = dict(n_layers=5, shapes=[(24, 256), (16, 128)], block=64, K=64, alpha=0.3)


def _layer_sums(orc, layer, cb):
    """Oracle round trip of the matrices of one layer -> (4 distortion sums, number of weights)."""
    total = np.zeros(4)
    n = 0
    for mid, (d_out, d_in) in enumerate(TINY["shapes"]):
        rng = np.random.default_rng(1000 + 16 * layer + mid)
        W = (rng.standard_t(4, (d_out, d_in)) * np.exp(0.7 * rng.standard_normal((d_out, 1)))).astype(np.float32)
        act = np.exp(rng.standard_normal(d_in)).astype(np.float32)
        s = orc.channel_scales(act, TINY["alpha"])
        signs = orc.make_signs(7, d_in)
        sigma, _ = orc.calibrate(W, TINY["block"], s, signs)
        enc = orc.encode(W, TINY["block"], cb, s, signs, sigma)
        what = orc.decode(enc["packed"], enc["row_norm"], TINY["block"], cb, s, signs, sigma, d_in)
        total += orc.distortion(W, what, act)
        n += d_out * d_in
    return total, n


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    sys.path.insert(0, os.path.join(ROOT, "tests"))
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from oracle import oracle as orc
    from paper_2605_26339_b200.model_codec import combine_distortion, shard_layers

    cb = load_golden_codebook(TINY["K"])
    mine = shard_layers(TINY["n_layers"], rank, world)
    sums, n = np.zeros(4), 0
    for layer in mine:
        s4, k = _layer_sums(orc, layer, cb)
        sums += s4
        n += k
    res = combine_distortion(torch.from_numpy(sums), n)
    # timing of a multi-rank run is the slowest rank's: the same MAX all-reduce the benchmark uses
    t = torch.tensor([10.0 + rank], dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    np.save(os.path.join(out_dir, f"rank{rank}.npy"),
            np.array([res["rho_w"], res["rho_o_diag"], res["mse"], res["n_weights"], float(t[0]), len(mine)]))
    dist.destroy_process_group()


def test_shard_layers_partition():
    from paper_2605_26339_b200.model_codec import shard_layers
    for n_layers, world in [(40, 8), (22, 4), (5, 2), (3, 4), (1, 1)]:
        parts = [shard_layers(n_layers, r, world) for r in range(world)]
        assert sorted(sum(parts, [])) == list(range(n_layers))           # every layer exactly once
        assert max(map(len, parts)) - min(map(len, parts)) <= 1          # balanced
    with pytest.raises(ValueError):
        shard_layers(4, 2, 2)


def test_two_ranks_reproduce_the_single_process_figures(orc, tmp_path):
    world, port = 2, 29500 + os.getpid() % 2000
    mp.start_processes(_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True, start_method="spawn")
    r0, r1 = (np.load(tmp_path / f"rank{r}.npy") for r in range(world))
    assert np.array_equal(r0[:5], r1[:5])            # both ranks hold the reduced figures
    assert r0[4] == 11.0                             # MAX over ranks
    assert r0[5] + r1[5] == TINY["n_layers"]
    cb = load_golden_codebook(TINY["K"])
    sums, n = np.zeros(4), 0
    for layer in range(TINY["n_layers"]):
        s4, k = _layer_sums(orc, layer, cb)
        sums += s4
        n += k
    assert r0[3] == n
    np.testing.assert_allclose(r0[0], np.sqrt(sums[0] / sums[1]), rtol=1e-12)
    np.testing.assert_allclose(r0[1], np.sqrt(sums[2] / sums[3]), rtol=1e-12)
    np.testing.assert_allclose(r0[2], sums[0] / n, rtol=1e-12)
