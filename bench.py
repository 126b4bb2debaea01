#!/usr/bin/env python
"""Benchmark of the QAM-W codec hot path on B200: calibrate -> encode -> decode -> distortion
over every linear weight of a synthetic Llama-2-13B-shaped model (configuration "cfg3").

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload cfgX]

One JSON line is printed by rank 0.  A "step" is one pass of the whole path over the model.
The step runs phase by phase over all matrices (all calibrations, then all encodes, ...), so
every phase streams a working set far larger than L2 (8.7 - 51 GB) and no L2 flush is needed.
`value` is whole-step throughput with inputs resident in HBM; `e2e` is the same step fed from
pinned host memory with the packed result read back; `--impl reference` times the CPU oracle.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "encode Gweights/s and decode GB/s (BF16 out) at 13B shapes; % of roofline"


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3")
    ap.add_argument("--layers", type=int, default=0, help="debug: only the first LAYERS layers")
    ap.add_argument("--K", type=int, default=0)
    ap.add_argument("--block", type=int, default=0)
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU work budget of the oracle baseline")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    return ap.parse_args()


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), "measured"
    except Exception:
        return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.rows = []
        self.proc = None
        self.gpu_index = gpu_index

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.gpu_index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                 "-lms", "100"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            parts = [p.strip() for p in r.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                power.append(float(parts[2]))
            except ValueError:
                continue
            for n, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": float(np.median(sm)), "sm_max_mhz": float(max(mx)), "reasons": sorted(reasons),
                "samples": len(sm), "power_w_max": max(power)}


# ----------------------------------------------------------------------------------------------
# oracle legs (cpu_baseline of our arm, and the whole reference arm)
# ----------------------------------------------------------------------------------------------
def oracle_sample_problem(spec, rows_a: int, rows_b: int, cb_host):
    """Rows of the two matrix classes of the workload (wide-out and wide-in), drawn on the CPU
    with the workload's recipe, with oracle-side metadata."""
    import torch
    from oracle import oracle as orc
    from paper_2605_26339_b200 import synth

    classes = sorted({(m.d_in) for m in spec.matrices})
    probs = []
    for d_in, rows in zip((classes[0], classes[-1]), (rows_a, rows_b)):
        if rows <= 0:
            continue
        m = synth.MatrixSpec(f"sample_{d_in}", rows, d_in)
        W = synth.make_weight(spec, m, spec.base_seed + d_in)
        Wb = W.view(torch.int16).numpy().view(np.uint16) if W.dtype == torch.bfloat16 else W.numpy()
        act = synth.make_act_rms(spec, d_in, spec.base_seed + d_in).numpy()
        s = orc.channel_scales(act, float(np.float32(spec.alpha))) if spec.alpha else None
        signs = orc.make_signs(0x51A5C0DEC0FFEE01, d_in)
        sigma, _ = orc.calibrate(Wb, spec.block, s, signs)
        probs.append(dict(W=Wb, s=s, signs=signs, sigma=sigma, d_in=d_in, rows=rows))
    return probs


def oracle_pass(spec, probs, cb_host) -> float:
    """Oracle encode + decode of the sample; returns seconds."""
    from oracle import oracle as orc

    t0 = time.perf_counter()
    for pr in probs:
        enc = orc.encode(pr["W"], spec.block, cb_host, pr["s"], pr["signs"], pr["sigma"])
        orc.decode(enc["packed"], enc["row_norm"], spec.block, cb_host, pr["s"], pr["signs"], pr["sigma"], pr["d_in"])
    return time.perf_counter() - t0


def size_oracle_sample(spec, cb_host, seconds: float):
    """Probe with a few rows, then size the sample for about `seconds` of wall time."""
    probe = oracle_sample_problem(spec, 256, 96, cb_host)
    oracle_pass(spec, probe, cb_host)  # first call builds / warms the library
    t = oracle_pass(spec, probe, cb_host)
    w = sum(p["rows"] * p["d_in"] for p in probe)
    rate = w / max(t, 1e-6)
    classes = sorted({m.d_in for m in spec.matrices})
    target = rate * seconds
    rows_a = max(32, int(0.7 * target / classes[0]))
    rows_b = max(16, int(0.3 * target / classes[-1])) if len(classes) > 1 else 0
    return rows_a, rows_b


def golden_or_trained_codebook(K: int):
    """Codebook for the oracle legs: trained by the oracle's own trainer at small size would take
    minutes, so the oracle-trained table stored with the tests is used when present."""
    path = os.path.join(ROOT, "tests", "golden", f"codebook_K{K}.txt")
    if os.path.exists(path):
        rows = []
        with open(path) as f:
            for line in f:
                if line.startswith("#") or not line.strip():
                    continue
                a, b = line.split()
                rows.append((int(a, 16), int(b, 16)))
        return np.array(rows, dtype=np.uint32).view(np.float32)
    from oracle import oracle as orc
    return orc.train_codebook(K, 1 << 16, 0, 30, 1e-5)[0]


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    from oracle import oracle as orc
    from paper_2605_26339_b200 import synth

    spec = synth.workload(args.workload, args.K or None, args.block or None)
    cb_host = golden_or_trained_codebook(spec.K)
    rows_a, rows_b = size_oracle_sample(spec, cb_host, min(args.cpu_seconds, 8.0))
    probs = oracle_sample_problem(spec, rows_a, rows_b, cb_host)
    n_w = sum(p["rows"] * p["d_in"] for p in probs)
    for _ in range(args.warmup):
        oracle_pass(spec, probs, cb_host)
    times = [oracle_pass(spec, probs, cb_host) for _ in range(args.steps)]
    t = float(np.mean(times))
    value = n_w / t / 1e9
    sample = f"{rows_a} rows of d_in={probs[0]['d_in']}" + (f" + {rows_b} rows of d_in={probs[-1]['d_in']}" if rows_b else "")
    out = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": "Gweights/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_label(spec), "sample": sample},
        "cpu_baseline": {"value": value, "unit": "Gweights/s", "cores": orc.num_threads(), "kind": "oracle",
                         "sample": sample + " per step, encode + decode"},
        "e2e": {"value": value, "unit": "Gweights/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(out), flush=True)


def workload_label(spec) -> str:
    shapes = ", ".join(f"{m.name}[{m.d_out},{m.d_in}]" for m in spec.matrices)
    return (f"{spec.name}: {spec.n_layers} layers x ({shapes}), {spec.w_dtype} weights, {spec.entry} entries, "
            f"K={spec.K}, block={spec.block}, alpha={spec.alpha}")


# ----------------------------------------------------------------------------------------------
# our arm
# ----------------------------------------------------------------------------------------------
def run_ours(args):
    import torch
    import torch.distributed as dist

    from paper_2605_26339_b200 import binding as q
    from paper_2605_26339_b200 import synth
    from paper_2605_26339_b200.model_codec import ModelCodec

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the codec has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    spec = synth.workload(args.workload, args.K or None, args.block or None)
    layers = list(range(min(args.layers, spec.n_layers))) if args.layers else None
    t0 = time.perf_counter()
    cb_host, train_mse = q.train_codebook(spec.K)
    train_host_s = time.perf_counter() - t0
    gpu_train = q.train_codebook_gpu(spec.K) if rank == 0 else None  # same rules on the device; timed, not used below
    mc = ModelCodec.from_synthetic(spec, dev, cb_host, rank=rank, layers=layers)
    n_w = mc.n_weights
    enc_bytes, dec_bytes = mc.algorithmic_bytes()
    phases = [("calibrate", mc.calibrate_all), ("encode", mc.encode_all), ("decode", mc.decode_all),
              ("distortion", mc.distortion_all)]

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()

    for _ in range(args.warmup):
        mc.step()
    barrier()
    sampler = ClockSampler("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
    if rank == 0:
        sampler.start()
        time.sleep(0.2)
    ev = [[(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in phases]
          for _ in range(args.steps)]
    barrier()
    t_wall = time.perf_counter()
    for k in range(args.steps):
        for (name, fn), (e0, e1) in zip(phases, ev[k]):
            e0.record()
            fn()
            e1.record()
    barrier()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop() if rank == 0 else None
    phase_ms = np.array([[e0.elapsed_time(e1) for (e0, e1) in ev[k]] for k in range(args.steps)]).mean(0)
    step_ms = float(ev[0][0][0].elapsed_time(ev[-1][-1][1]) / args.steps)  # device time incl. gaps between phases
    t = torch.tensor([step_ms, *phase_ms.tolist()], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    step_ms, cal_ms, enc_ms, dec_ms, dis_ms = t.cpu().tolist()
    status_word = int(mc.status.cpu()[0])
    totals = mc.totals()

    # ---- end-to-end: inputs in pinned host memory, packed stream read back -----------------------
    e2e = e2e_full = None
    if not args.no_e2e:
        e2e = run_e2e(mc, args, world, dist if world > 1 else None)
        if world == 1:
            e2e_full = run_e2e(mc, args, world, None, with_reconstruction=True)

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    peak, peak_kind = measured_peaks()
    enc_launches = len({mc._encoder_class(s.d_in) for s in mc.slots}) if mc.use_batch else len(mc.slots)
    dec_launches = 1 if mc.use_batch else len(mc.slots)
    fp32_peak = q.measure_fp32_peak()
    pipe = load_pipe_note()
    enc_gbs = enc_bytes / (enc_ms * 1e-3) / 1e9
    dec_gbs = dec_bytes / (dec_ms * 1e-3) / 1e9
    out = {
        "metric": METRIC,
        "value": world * n_w / (step_ms * 1e-3) / 1e9,
        "unit": "Gweights/s",
        "n_gpus": world, "steps": args.steps, "warmup": args.warmup, "ms_per_step": step_ms,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": workload_label(spec), "weights_per_gpu": n_w, "matrices": len(mc.slots), "streams": mc.n_streams,
                   "l2": "no flush: every phase streams 8.7-51 GB per step, far more than the 126 MB L2",
                   "step": "calibrate + encode + decode + distortion, phase by phase over all matrices",
                   "table": {"grid": int(mc.codebook.table_info()[0]), "bytes": int(mc.codebook.table_info()[5])},
                   "codebook_train_mse": train_mse},
        "codebook_training": {"K": spec.K, "samples": 1 << 20, "host_s": train_host_s,
                              "device_s": gpu_train["seconds"], "device_updates": gpu_train["iters"],
                              "device_vs_host_max_abs_diff": float(np.abs(gpu_train["codebook"] - cb_host).max()),
                              "paper": "about 5 s per bitrate level, hardware not stated (Limitations section)"},
        "fp32_issue_peak": {"lane_inst_per_s": fp32_peak, "tflops_as_fma": 2 * fp32_peak / 1e12,
                            "how": "qamw_measure_fp32_peak: FMA kernel, eight independent chains per thread"},
        "encode_gweights_s": world * n_w / (enc_ms * 1e-3) / 1e9,
        "decode_gb_s": world * dec_gbs,
        "phases_ms": {"calibrate": cal_ms, "encode": enc_ms, "decode": dec_ms, "distortion": dis_ms},
        "clocks": clocks,
        "gpu_launches": mc.kernel_launches_per_step() * args.steps,
        "roofline": {"kernel": "encode2_kernel", "bound": "hbm", "achieved": enc_gbs, "peak": peak, "unit": "GB/s",
                     "frac": enc_gbs / peak, "peak_kind": f"of {peak_kind}", "frac_of_nominal_8TBs": enc_gbs / 8000.0,
                     "algorithmic_bytes_per_launch": enc_bytes / enc_launches, "avg_launch_ms": enc_ms / enc_launches,
                     "launches_per_step": enc_launches, "traffic": None},
        "roofline_decode": {"kernel": "decode2_kernel", "bound": "hbm", "achieved": dec_gbs, "peak": peak,
                            "unit": "GB/s", "frac": dec_gbs / peak, "peak_kind": f"of {peak_kind}",
                            "frac_of_nominal_8TBs": dec_gbs / 8000.0,
                            "algorithmic_bytes_per_launch": dec_bytes / dec_launches, "avg_launch_ms": dec_ms / dec_launches,
                            "launches_per_step": dec_launches, "traffic": None},
        "quality": totals, "status_word": status_word, "wall_s_timed_region": t_wall,
    }
    out["fused_gemv"] = time_fused_gemv(mc, peak)
    out["graph_step_ms"] = time_graph_step(mc, args.steps)
    out["polar_baseline"] = time_polar_encode(mc)
    if e2e is not None:
        out["e2e"] = e2e
    if e2e_full is not None:
        out["e2e_with_reconstruction"] = e2e_full
    if not args.no_cpu_baseline and world == 1:
        out["cpu_baseline"] = cpu_baseline(spec, golden_or_trained_codebook(spec.K), args)
    traffic = load_traffic_note()
    if traffic:  # measured bytes per weight x weights of the average launch
        out["roofline"]["traffic"] = traffic["encode"] * n_w / enc_launches
        out["roofline_decode"]["traffic"] = traffic["decode"] * n_w / dec_launches
    if pipe and clocks and clocks.get("sm_mhz"):
        # The encoder is bound by the shared-memory / load-store data pipe, not by HBM: one wavefront per
        # clock per SM is that pipe's peak, and ncu counted how many wavefronts a 2-D point costs.
        sms = torch.cuda.get_device_properties(dev).multi_processor_count
        wf_s = pipe["encode_lsu_wavefronts_per_point"] * (n_w / 2) / (enc_ms * 1e-3)
        pk = sms * clocks["sm_mhz"] * 1e6
        out["roofline_encode_pipe"] = {"kernel": "encode2_kernel", "bound": "lsu (shared-memory data pipe)",
                                       "achieved": wf_s / 1e9, "peak": pk / 1e9, "unit": "Gwavefronts/s",
                                       "frac": wf_s / pk, "wavefronts_per_point": pipe["encode_lsu_wavefronts_per_point"],
                                       "source": "profiles/encode_pipe.txt (ncu l1tex__data_pipe_lsu_wavefronts)"}
    print(json.dumps(out), flush=True)
    if world > 1:
        dist.destroy_process_group()


def time_polar_encode(mc, calls=5):
    """The polar baseline quantiser of Section 3.5 (Rayleigh Lloyd-Max amplitude x uniform phase, same bits per
    pair as the workload's codebook, split 5 + 6 at eleven bits) through the same encoder kernel, on the
    matrices of the first layer, into scratch outputs."""
    import torch

    from paper_2605_26339_b200 import binding as q
    B = int(np.log2(mc.spec.K))
    Ba = B // 2
    Bp = B - Ba
    slots = mc.slots[:7]
    try:
        levels, _ = q.polar_train(Ba)
        cb = q.Codebook.polar(levels, Ba, Bp)
        outs = [(torch.empty_like(s.packed), torch.empty_like(s.row_norm)) for s in slots]

        batch = q.Batch([q.make_matrix(s.params, s.W, s.chan_scale, s.signs, s.sigma, s.act_rms, pk, rn, s.w_hat, s.dist)
                         for s, (pk, rn) in zip(slots, outs)], cb)

        def run():
            batch.encode(mc.status)

        run()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(calls):
            run()
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / calls
        n_w = sum(s.d_out * s.d_in for s in slots)
        return {"amplitude_bits": Ba, "phase_bits": Bp, "matrices": len(slots), "encode_ms": ms,
                "encode_gweights_s": n_w / (ms * 1e-3) / 1e9, "note": "batched launches, as the 2-D codec"}
    except Exception as exc:  # noqa: BLE001 - a side figure: reported, not fatal
        sys.stderr.write(f"polar baseline timing failed: {exc}\n")
        return None


def time_graph_step(mc, steps):
    """The same step replayed as one CUDA graph (what a launch-bound small model should use); None if the
    step cannot be captured."""
    import torch

    try:
        graph = mc.capture_step()
        for _ in range(3):
            graph.replay()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(steps):
            graph.replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / steps
    except Exception as exc:  # noqa: BLE001 - reported, not fatal: the eager timing above is the benchmark
        sys.stderr.write(f"graph capture of the step failed: {exc}\n")
        return None


def time_fused_gemv(mc, peak_gbs, calls=50):
    """y = W_hat x straight from the packed stream (qamw_decode_gemv), one activation vector, every matrix of the
    first layer in turn so that the packed bytes of a round exceed L2; beside it the paper's pipeline on the same
    matrices: a bf16 product on the already decoded W_hat (what follows qamw_decode there)."""
    import torch

    from paper_2605_26339_b200 import binding as q
    slots = [s for s in mc.slots if s.d_in % 32 == 0][:7]
    if not slots:
        return None
    dev = mc.device
    xs = [torch.randn((1, s.d_in), device=dev) for s in slots]
    ys = [torch.empty((s.d_out, 1), device=dev) for s in slots]
    xb = [x.to(torch.bfloat16).T.contiguous() for x in xs]
    ws = torch.empty(max(4 * s.d_in for s in slots) + 64, dtype=torch.uint8, device=dev)

    def fused():
        for s, x, y in zip(slots, xs, ys):
            q.decode_gemv(s.packed, s.row_norm, s.chan_scale, s.signs, s.sigma, mc.codebook, s.params, x, y, ws)

    def bf16():
        for s, x in zip(slots, xb):
            torch.matmul(s.w_hat, x)

    def timed(fn):
        for _ in range(3):
            fn()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        torch.cuda.synchronize()
        e0.record()
        for _ in range(calls):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / calls * 1e3  # microseconds per round

    t_fused, t_bf16 = timed(fused), timed(bf16)
    B = int(np.log2(mc.spec.K))
    packed_bytes = sum(s.d_out * s.d_in * B / 16 for s in slots)
    return {"matrices": [[s.d_out, s.d_in] for s in slots], "vectors": 1, "us_per_round": t_fused,
            "packed_gb_s": packed_bytes / t_fused / 1e3, "frac_of_hbm_peak": packed_bytes / t_fused / 1e3 / peak_gbs,
            "bf16_product_on_decoded_us": t_bf16, "kernel_launches_per_round": len(slots),
            "note": "bound by the shared-memory gather of one codeword per pair, not by HBM"}


def load_traffic_note():
    """DRAM bytes per weight measured once with ncu on the cfg4 matrix (profiles/dram_traffic.txt:
    `key value` lines).  The note carries the hash of the kernel source it was taken from; if the
    kernels have changed since, the traffic is unknown again (None)."""
    import hashlib
    try:
        note = {}
        with open(os.path.join(ROOT, "profiles", "dram_traffic.txt")) as f:
            for line in f:
                if line.strip() and not line.startswith("#"):
                    k, v = line.split()[:2]
                    note[k] = v
        src = os.path.join(ROOT, "paper_2605_26339_b200", "csrc", "qamw_rows.cu")
        with open(src, "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != note.get("kernel_source_sha256"):
                return None
        return {"encode": float(note["encode_dram_bytes_per_weight"]),
                "decode": float(note["decode_dram_bytes_per_weight"])}
    except Exception:
        return None


def load_pipe_note():
    """Load/store-pipe wavefronts per 2-D point of the encoder, counted once with ncu
    (profiles/encode_pipe.txt, same format and staleness rule as the traffic note)."""
    import hashlib
    try:
        note = {}
        with open(os.path.join(ROOT, "profiles", "encode_pipe.txt")) as f:
            for line in f:
                if line.strip() and not line.startswith("#"):
                    k, v = line.split()[:2]
                    note[k] = v
        with open(os.path.join(ROOT, "paper_2605_26339_b200", "csrc", "qamw_rows.cu"), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != note.get("kernel_source_sha256"):
                return None
        return {"encode_lsu_wavefronts_per_point": float(note["encode_lsu_wavefronts_per_point"])}
    except Exception:
        return None


def run_e2e(mc, args, world, dist, with_reconstruction=False):
    """The same step driven from pinned host memory: every matrix is copied host -> device, then
    calibrated, encoded, decoded and scored; the packed stream, row norms and distortion sums are
    copied back.  Copies run on their own streams and overlap the kernels."""
    import psutil
    import torch

    dev = mc.device
    slots = mc.slots
    per_layer = len(mc.spec.matrices)
    n_layers = len(slots) // per_layer
    layer_bytes = sum(s.W.numel() * s.W.element_size() for s in slots[:per_layer])
    avail = psutil.virtual_memory().available
    host_layers = max(1, min(n_layers, int(0.35 * avail / max(1, world) / layer_bytes)))  # all ranks share the host
    host_W = []
    for s in slots[: host_layers * per_layer]:
        h = torch.empty(s.W.shape, dtype=s.W.dtype, pin_memory=True)
        h.copy_(s.W)
        host_W.append(h)
    out_bufs = {}
    for s in slots[:per_layer]:
        out_bufs[(s.d_out, s.d_in)] = (torch.empty(s.packed.shape, dtype=torch.uint8, pin_memory=True),
                                       torch.empty(s.row_norm.shape, dtype=torch.float32, pin_memory=True))
    what_bufs = {}
    if with_reconstruction:
        for s in slots[:per_layer]:
            what_bufs[(s.d_out, s.d_in)] = torch.empty(s.w_hat.shape, dtype=torch.bfloat16, pin_memory=True)
    dist_host = torch.empty((len(slots), 4), dtype=torch.float64, pin_memory=True)
    h2d, comp, d2h = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)
    h2d_bytes = sum(s.W.numel() * s.W.element_size() for s in slots)
    d2h_bytes = sum(s.packed.numel() + 4 * s.row_norm.numel() + 32 for s in slots)
    if with_reconstruction:
        d2h_bytes += sum(2 * s.w_hat.numel() for s in slots)

    def one_step():
        for i, s in enumerate(slots):
            src = host_W[i % len(host_W)]
            with torch.cuda.stream(h2d):
                s.W.copy_(src, non_blocking=True)
                ready = h2d.record_event()
            with torch.cuda.stream(comp):
                comp.wait_event(ready)
                from paper_2605_26339_b200 import binding as q
                q.calibrate(s.W, s.params, s.chan_scale, s.signs, s.sigma, mc.workspace, mc.status)
                q.encode(s.W, s.params, s.chan_scale, s.signs, s.sigma, mc.codebook, s.packed, s.row_norm, mc.status)
                q.decode(s.packed, s.row_norm, s.chan_scale, s.signs, s.sigma, mc.codebook, s.params, s.w_hat)
                q.distortion(s.W, s.w_hat, s.act_rms, s.params, s.dist)
                done = comp.record_event()
            with torch.cuda.stream(d2h):
                d2h.wait_event(done)
                pk, nm = out_bufs[(s.d_out, s.d_in)]
                pk.copy_(s.packed, non_blocking=True)
                nm.copy_(s.row_norm, non_blocking=True)
                dist_host[i].copy_(s.dist, non_blocking=True)
                if with_reconstruction:
                    what_bufs[(s.d_out, s.d_in)].copy_(s.w_hat, non_blocking=True)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()

    one_step()
    barrier()
    steps = max(1, min(args.steps, 2 if with_reconstruction else 3))
    t0 = time.perf_counter()
    for _ in range(steps):
        one_step()
    barrier()
    sec = (time.perf_counter() - t0) / steps
    t = torch.tensor([sec], dtype=torch.float64, device=dev)
    if dist is not None:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    sec = float(t.cpu()[0])
    return {"value": world * mc.n_weights / sec / 1e9, "unit": "Gweights/s", "h2d_bytes_per_step": h2d_bytes,
            "d2h_bytes_per_step": d2h_bytes, "ms_per_step": sec * 1e3, "steps": steps, "host_layers": host_layers,
            "note": ("weights from pinned host memory; packed stream, row norms, distortion sums and the decoded bf16 "
                     "matrices read back" if with_reconstruction else
                     "encode side end to end: weights from pinned host memory; packed stream, row norms and distortion "
                     "sums read back; the bf16 reconstruction stays on the device, where the paper's pipeline consumes "
                     "it (e2e_with_reconstruction also copies it back)")}


def cpu_baseline(spec, cb_host, args):
    from oracle import oracle as orc

    rows_a, rows_b = size_oracle_sample(spec, cb_host, args.cpu_seconds)
    probs = oracle_sample_problem(spec, rows_a, rows_b, cb_host)
    n_w = sum(p["rows"] * p["d_in"] for p in probs)
    t = oracle_pass(spec, probs, cb_host)
    sample = f"{rows_a} rows of d_in={probs[0]['d_in']}" + (f" + {rows_b} rows of d_in={probs[-1]['d_in']}" if rows_b else "")
    return {"value": n_w / t / 1e9, "unit": "Gweights/s", "cores": orc.num_threads(), "kind": "oracle",
            "sample": sample + ", oracle encode + decode, once", "seconds": t}


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
