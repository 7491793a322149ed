#!/usr/bin/env python
"""Benchmark of the HIGGS quantized linear layer on B200.

One "step" = one decode pass (Appendix F: rotate activations, stream codes, table lookup, contraction, reduce)
over the seven linear layers of one Llama-shaped transformer block for one batch of synthetic activations, wired as
in the block: q, k, v read one input (rotated once), o its own, gate and up one (rotated once), down its own.  The headline value is the
effective weight bandwidth (packed codes + scales bytes of the layer set / time per step).  The encoder
(Algorithm 1) and the grid fit (Algorithm 2) run once during set-up, on the GPU, and are reported separately.

The default workload is the largest single-GPU configuration: the Llama-3.1-70B layer shapes with the seeded 3/4-bit
assignment (3.5 bits per weight on average), batch 1.  The same run reports, under "detail", one row per layer, grid
and batch of the other configurations (8B shapes at three grids and batches 1/4/16, and at batches 64/256 with
log-normal channel scales; 1B shapes at batches 1/16), each with its share of the roofline and a parity check of the
timed output against the fp64 oracle on sampled rows.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama-3.1-70b] [--batch 1] [--grid mixed]
    python bench.py --impl reference ...      # the fp64 CPU oracle timed on the host cores (reported baseline)

Under torchrun (N > 1) every rank runs an independent replica of the same layer set on its own GPU (the layer
needs no collective); the reported value is the sum over ranks divided by the slowest rank's time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from synth import inputs  # noqa: E402

G = 1024
L2_BYTES = 126 * 1024 * 1024


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="llama-3.1-70b", choices=list(inputs.LAYER_SETS))
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--grid", default=None,
                    help="p,n for every layer, or 'mixed': 3 or 4 bits per matrix (p=2 n=64 / n=256) from the seeded assignment "
                         "averaging 3.5 bits (the default for the Llama-3.1-70B shapes; the other sets default to 2,256)")
    ap.add_argument("--no-graph", action="store_true", help="launch kernels directly instead of replaying CUDA graphs")
    ap.add_argument("--steps-per-graph", type=int, default=8,
                    help="at most this many consecutive steps (over rotating weight copies) per CUDA graph; the largest divisor "
                         "of --steps not above it is used, so that exactly --steps steps run from equal graphs")
    ap.add_argument("--shard", choices=["none", "rows", "k"], default="none",
                    help="none: every rank runs an independent replica (the default); rows / k: ONE layer set sharded over the "
                         "ranks by rows (outputs written into every rank's buffer from the kernels' epilogues) or along K on "
                         "group boundaries (partial outputs into every rank's slot buffer, then a slot-ordered sum), through "
                         "peer-mapped symmetric memory")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-detail", action="store_true", help="skip the per-layer rows and the rows of the other configurations")
    args = ap.parse_args()
    if args.grid is None:
        args.grid = "mixed" if args.workload == "llama-3.1-70b" else "2,256"
    return args


def layer_bytes(N, K, p, n):
    bits = {(2, 256): 4, (1, 16): 4, (2, 64): 3, (2, 16): 2, (1, 8): 3, (1, 4): 2, (1, 256): 8}[(p, n)]
    return N * K * bits // 8 + N * (K // G) * 2


def layer_grids(args, layers, cfg):
    """(p, n) per layer: one grid for all, or the block of the seeded 3/4-bit assignment closest to 3.5 bits."""
    if args.grid != "mixed":
        p, n = (int(v) for v in args.grid.split(","))
        return [(p, n)] * len(layers), f"p={p} n={n}"
    blocks = inputs.bitwidth_assignment(7000 + cfg, layers)
    sizes = np.array([N * K for _, N, K in layers], dtype=np.float64)
    best = min(blocks, key=lambda b: abs(float((np.array(b) * sizes).sum() / sizes.sum()) - 3.5))
    mean = float((np.array(best) * sizes).sum() / sizes.sum())
    pn = [(2, 64) if b == 3 else (2, 256) for b in best]
    return pn, "mixed " + ",".join(f"{nm}:{b}" for (nm, _, _), b in zip(layers, best)) + f" bits ({mean:.2f} bits/weight)"


def algorithmic_bytes(N, K, p, n, B):
    """codes + scales + activations in + outputs out + grid table (per launch of the product kernel)."""
    return layer_bytes(N, K, p, n) + B * K * 2 + B * N * 4 + n * p * 4


def measured_peaks():
    """(HBM GB/s, dense 16-bit tensor TFLOP/s burst, source) from the generated file, else the stated fallback."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            d = json.load(f)
        return float(d["hbm_gbs"]), float(d["bf16_tflops"]), "measured"
    except Exception:
        return 6650.0, 1590.0, "fallback"


# Encoder rooflines.  ALU: the pruned search is bound by instruction issue (profiles/encode_pruned_kernel_...): ncu
# counted 3748 warp instructions per (row, group) task of 1024 weights for p=2 n=256 (smsp__inst_executed.sum / tasks);
# achieved = weights/s x that count, against 148 SMs x 4 schedulers x 1 warp instruction per clock.  It is derived from
# the measured weights/s and a counted constant, not read from a counter in this run.  HBM: what the encoder must move
# per weight - the bf16 weight in, log2(n)/p bits of code and 16/1024 bits of scale out - against the copy peak; this
# is the floor an exact pruned search approaches.
ENCODER_WARP_INSTR_PER_WEIGHT = {(2, 256): 1776.0 / 1024.0}


def encoder_rooflines(weights_per_s, pn, sizes, clocks, hbm_peak, peak_src):
    out = []
    bits = {(2, 256): 4, (1, 16): 4, (2, 64): 3, (2, 16): 2, (1, 8): 3, (1, 4): 2, (1, 256): 8}
    total = float(sum(sizes))
    bytes_per_weight = sum(s * (2.0 + bits[k] / 8.0 + 2.0 / G) for s, k in zip(sizes, pn)) / total
    gbs = weights_per_s * bytes_per_weight / 1e9
    out.append({"bound": "hbm", "achieved": gbs, "peak": hbm_peak, "unit": "GB/s", "frac": gbs / hbm_peak,
                "bytes_per_weight": bytes_per_weight, "peak_source": f"of {peak_src}"})
    grids = set(pn)
    if len(grids) == 1 and next(iter(grids)) in ENCODER_WARP_INSTR_PER_WEIGHT:
        ipw = ENCODER_WARP_INSTR_PER_WEIGHT[next(iter(grids))]
        mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
        peak = 148 * 4 * mhz * 1e6 / 1e9                    # G warp instructions / s
        achieved = weights_per_s * ipw / 1e9
        out.append({"bound": "alu", "achieved": achieved, "peak": peak, "unit": "G warp-instr/s", "frac": achieved / peak,
                    "warp_instr_per_weight": ipw,
                    "note": "derived: measured weights/s of whole higgs_quantize calls x warp instructions per weight "
                            "counted by ncu in the committed capture, against the issue rate of 148 SMs x 4 schedulers"})
    return out


def max_over_ranks(ms: float, device, world: int) -> float:
    """Duration of the timed region as the slowest rank saw it (replicas run independently; no data-path collective)."""
    if world <= 1:
        return float(ms)
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def aggregate_value(bytes_per_step: int, steps: int, ms: float, world: int) -> float:
    """Whole-job effective weight bandwidth in GB/s: every rank processed bytes_per_step per step."""
    return world * bytes_per_step / (ms / steps * 1e-3) / 1e9


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits", "-lms", "100"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.strip().splitlines():
            f = [c.strip() for c in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1]))
                mx.append(float(f[2]))
            except ValueError:
                continue
            for nm, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


# --------------------------------------------------------------------------------------------- reference arm
def oracle_sample(layers, pn, cfg, xi, grids64, B, rows):
    """`rows` rows of every layer, encoded by the oracle (rows are independent, so this is a plain sample of the set)."""
    import oracle
    sample = []
    for li, (name, N, K) in enumerate(layers):
        r = min(rows, N)
        W = inputs.make_weights(r, K, inputs.weight_seed(cfg, li), bf16=True).astype(np.float64)
        q = oracle.quantize(W, G, grids64[pn[li]], xi)
        sc = oracle.round_scales_fp16(q.scales).astype(np.float64)
        x = inputs.make_activations(B, K, inputs.activation_seed(cfg, B) + li).astype(np.float64)
        sample.append((W, q.codes, sc, x, r, K, pn[li]))
    return sample


def run_reference(args):
    """The fp64 oracle (as it stands) on the host cores: the same metric on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from synth import grids as stored_grids

    layers = inputs.LAYER_SETS[args.workload]
    cfg = inputs.CONFIG_OF_SET[args.workload]
    pn, grid_text = layer_grids(args, layers, cfg)
    xi = inputs.rht_seed(cfg)
    grids64 = {k: stored_grids.load(*k) for k in set(pn)}
    B = args.batch
    rows = 16 if args.workload == "llama-3.1-70b" else 64
    sample = oracle_sample(layers, pn, cfg, xi, grids64, B, rows)
    nbytes = sum(layer_bytes(r, K, *k) for *_, r, K, k in sample)

    def step():
        for _, codes, sc, x, r, K, k in sample:
            oracle.linear_dense(x, codes, sc, G, grids64[k], xi)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = (time.perf_counter() - t0) / max(args.steps, 1)
    value = nbytes / dt / 1e9
    desc = f"{rows} rows of each of the {len(layers)} layers per step (rows are independent), dequantise + fp64 matmul"
    line = {
        "impl": "reference", "metric": "higgs_linear_effective_weight_bandwidth", "value": value, "unit": "GB/s",
        "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": f"{args.workload} layer set ({len(layers)} matrices), grid {grid_text}, g=1024, batch {B}", "sample": desc},
        "cpu_baseline": {"value": value, "unit": "GB/s", "cores": oracle.threads(), "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def cpu_baseline(layers, pn, cfg, xi, grids64, B):
    """The oracle as it stands on this machine's cores, on a bounded row sample: the product (dequantise + fp64 matmul) on
    all cores and on one, and the encoder (Algorithm 1) likewise.  About 25 s in all."""
    import oracle
    cores = oracle.threads()
    rows = 64 if sum(N * K for _, N, K in layers) > 5e8 else 256
    smp = oracle_sample(layers, pn, cfg, xi, grids64, B, rows)
    nb = sum(layer_bytes(r, K, *k) for *_, r, K, k in smp)
    nw = sum(r * K for *_, r, K, k in smp)

    def product():
        for _, codes, sc, x, r, K, k in smp:
            oracle.linear_dense(x, codes, sc, G, grids64[k], xi)

    def encode():
        for W, _, _, _, r, K, k in smp:
            oracle.quantize(W, G, grids64[k], xi)

    def timed(fn, budget):
        reps, t0 = 0, time.perf_counter()
        while reps < 1 or time.perf_counter() - t0 < budget:
            fn()
            reps += 1
        return (time.perf_counter() - t0) / reps, reps

    dt_all, reps = timed(product, 8.0)
    dtq_all, _ = timed(encode, 4.0)
    oracle.set_threads(1)
    try:
        dt_one, _ = timed(product, 5.0)
        dtq_one, _ = timed(encode, 4.0)
    finally:
        oracle.set_threads(cores)
    return {"value": nb / dt_all / 1e9, "unit": "GB/s", "cores": cores, "kind": "oracle",
            "sample": f"{rows} rows of each of the {len(layers)} layers (rows are independent), dequantise + fp64 matmul, {reps} passes",
            "single_thread_value": nb / dt_one / 1e9,
            "quantize_weights_per_s": nw / dtq_all, "quantize_weights_per_s_single_thread": nw / dtq_one}


# --------------------------------------------------------------------------------------------- our arm: helpers
def divisor_at_most(steps: int, cap: int) -> int:
    """Largest divisor of `steps` that is <= cap (>= 1): `steps` steps then run from steps / d equal graphs."""
    for d in range(max(1, min(cap, steps)), 0, -1):
        if steps % d == 0:
            return d
    return 1


class Quantized:
    """One layer encoded on the device (Algorithm 1) with everything a timed product or a parity check needs."""

    def __init__(self, hb, torch, dev, name, N, K, pn, xi, grid, W, table=None):
        self.name, self.N, self.K, self.pn = name, N, K, pn
        self.desc = hb.make_desc(pn[0], pn[1], N, K, xi)
        self.grid, self.table = grid, table
        self.wsq = torch.empty(hb.higgs_workspace_bytes(self.desc, hb.HIGGS_OP_QUANTIZE), dtype=torch.uint8, device=dev)
        pk, sc, _ = hb.higgs_quantize(self.desc, W, grid, workspace=self.wsq, table=table)
        self.packed, self.scales = [pk], [sc]
        self.bytes = layer_bytes(N, K, *pn)

    def encode_again(self, hb, W):
        """A second call into the same buffers: only the library's kernels are inside a timed region around it."""
        hb.higgs_quantize(self.desc, W, self.grid, workspace=self.wsq, out=(self.packed[0], self.scales[0]), table=self.table)

    @classmethod
    def from_buffers(cls, name, desc, grid, packed, scales):
        """A layer whose packed buffers exist already (row-concatenated layers)."""
        q = cls.__new__(cls)
        q.name, q.N, q.K, q.pn, q.desc, q.grid = name, desc.N, desc.K, (desc.p, desc.n), desc, grid
        q.packed, q.scales, q.bytes, q.table, q.wsq = list(packed), list(scales), layer_bytes(desc.N, desc.K, desc.p, desc.n), None, None
        return q

    def ensure_copies(self, count):
        while len(self.packed) < count:
            self.packed.append(self.packed[0].clone())
            self.scales.append(self.scales[0].clone())


def parity_on_sampled_rows(hb, oracle, q, x_host32, y, xi, grid64, rows=16, seed=1):
    """The timed output against the fp64 oracle on `rows` sampled rows, given the device's own codes and stored scales:
    (max |dy| / max |y^|, max |dy| / rms(y^)) over the sample."""
    rng = np.random.default_rng(seed + q.N)
    ridx = np.sort(rng.choice(q.N, size=min(rows, q.N), replace=False))
    canon = hb.higgs_unpack_codes(q.desc, q.packed[0])
    codes = canon[ridx.tolist()].cpu().numpy().astype(np.int64)
    sc = hb.scales_from_tile_major(q.scales[0], q.N)[ridx.tolist()].float().cpu().numpy().astype(np.float64)
    del canon
    y_ref = oracle.linear_dense(x_host32.astype(np.float64), codes, sc, G, grid64, xi)
    got = y.float()[:, ridx.tolist()].cpu().numpy().astype(np.float64)
    err = np.max(np.abs(got - y_ref))
    return float(err / np.max(np.abs(y_ref))), float(err / np.sqrt(np.mean(y_ref ** 2)))


def time_product(hb, torch, stream, q, B, x_dev, reps=200, copies_bytes=512 << 20):
    """One launch of the product kernel (D2-D5 on already rotated activations) of layer `q` at batch B, timed with CUDA
    events on the launching stream: a CUDA graph of back-to-back launches over rotating weight copies (>= 512 MB, so no
    launch finds its codes in L2), every replay timed separately.  Returns mean / median / min microseconds per launch
    over the replays, the kernels per call and the output of the last launch."""
    d = q.desc
    xdag = hb.higgs_rotate_activations(d, x_dev)
    yk = torch.empty((B, d.N), dtype=torch.float32, device=x_dev.device)
    wk = torch.empty(hb.higgs_workspace_bytes(d, hb.HIGGS_OP_LINEAR, B), dtype=torch.uint8, device=x_dev.device)
    q.ensure_copies(min(1024, max(2, -(-copies_bytes // q.bytes))))
    n = len(q.packed)
    ev = lambda: torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        hb.higgs_linear_prerotated(d, xdag, q.packed[0], q.scales[0], q.grid, workspace=wk, y=yk, B=B)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for c in range(n):
                hb.higgs_linear_prerotated(d, xdag, q.packed[c], q.scales[c], q.grid, workspace=wk, y=yk, B=B)
        rounds = max(3, reps // n)
        for _ in range(3):
            g.replay()
        stream.synchronize()
        marks = [ev() for _ in range(rounds + 1)]
        marks[0].record(stream)
        for r in range(rounds):
            g.replay()
            marks[r + 1].record(stream)
        stream.synchronize()
    per = [marks[r].elapsed_time(marks[r + 1]) * 1e3 / n for r in range(rounds)]
    total = marks[0].elapsed_time(marks[rounds]) * 1e3 / (rounds * n)
    return {"us": total, "us_median": statistics.median(per), "us_min": min(per), "launches": rounds * n,
            "kernels_per_call": hb.higgs_linear_launch_count(d, B) - 1, "y": yk}


def product_row(hb, q, B, t, peak, peak_tf, parity=None):
    """A detail row: time, weight bandwidth and the roofline share of one layer at one batch."""
    p, n = q.pn
    tiled = hb.higgs_rotated_layout(q.desc, B) > 0
    alg = algorithmic_bytes(q.N, q.K, p, n, B)
    row = {"layer": q.name, "shape": f"{q.N}x{q.K}", "grid": f"p={p} n={n}", "B": B,
           "kernel": "linear_tc_kernel" if tiled else "linear_stream_kernel",
           "us": round(t["us"], 3), "us_median": round(t["us_median"], 3), "us_min": round(t["us_min"], 3),
           "weight_GBps": round(q.bytes / t["us"] / 1e3, 1)}
    if B >= 64 and tiled:
        tf = 2.0 * B * q.N * q.K / (t["us"] * 1e-6) / 1e12
        row["roofline"] = {"bound": "tensor", "achieved": round(tf, 1), "peak": peak_tf, "unit": "TFLOP/s", "frac": round(tf / peak_tf, 4)}
    else:
        gb = alg / (t["us"] * 1e-6) / 1e9
        row["roofline"] = {"bound": "hbm", "achieved": round(gb, 1), "peak": peak, "unit": "GB/s", "frac": round(gb / peak, 4)}
        # table lookups alone as a share of one 32-lane shared-memory wavefront per SM and clock (148 SMs, 1965 MHz)
        per_lookup = {(2, 256): 2, (2, 64): 2, (1, 16): 2, (1, 8): 2, (2, 16): 4, (1, 4): 4, (1, 256): 1}[(p, n)]
        row["lut_gather_frac"] = round(q.N * q.K / per_lookup / 32.0 / (t["us"] * 1e-6) / (148 * 1965e6), 4)
    if parity is not None:
        row["parity_max_rel"], row["parity_max_over_rms"] = (float(f"{v:.3g}") for v in parity)
    return row


def launch_floor(hb, torch, stream, blocks, threads, smem, reps=2000):
    """Microseconds per launch of a chain of kernels that do nothing, launched like the product kernels."""
    with torch.cuda.stream(stream):
        hb.higgs_launch_floor(blocks, threads, smem)
        stream.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=stream):
            for _ in range(50):
                hb.higgs_launch_floor(blocks, threads, smem)
        g.replay()
        stream.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(reps // 50):
            g.replay()
        b.record(stream)
        stream.synchronize()
    return a.elapsed_time(b) * 1e3 / (reps // 50 * 50)


def other_configurations(hb, torch, oracle, dev, stream, peak, peak_tf, fit_grid):
    """Rows for the configurations that are not the headline workload: the distinct layer shapes of the 8B set at three
    grids and batches 1, 4, 16; the same shapes at p=2 n=256 and batches 64, 256 with one log-normal scale per input
    channel; the 1B shapes at batches 1 and 16.  Every row carries the parity of its timed output on sampled rows."""
    rows = []
    plan = [("llama-3.1-8b", [(2, 256), (2, 64), (1, 16)], [1, 4, 16], False),
            ("llama-3.1-8b", [(2, 256)], [64, 256], True),
            ("llama-3.2-1b", [(2, 256)], [1, 16], False)]
    cache = {}
    for workload, grid_list, batches, lognormal in plan:
        cfg = inputs.CONFIG_OF_SET[workload] + (1 if lognormal else 0)      # configs[3] is the 8B set in the tensor regime
        xi = inputs.rht_seed(cfg)
        layers = inputs.LAYER_SETS[workload]
        seen = set()
        for li, (name, N, K) in enumerate(layers):
            if (N, K) in seen:
                continue
            seen.add((N, K))
            key = (workload, N, K)
            if key not in cache:
                cache[key] = torch.from_numpy(inputs.make_weights(N, K, inputs.weight_seed(inputs.CONFIG_OF_SET[workload], li),
                                                                  bf16=True)).to(dev).to(torch.bfloat16)
            W = cache[key]
            for pn in grid_list:
                grid = fit_grid(pn)
                q = Quantized(hb, torch, dev, name, N, K, pn, xi, grid, W)
                g64 = grid.cpu().numpy().astype(np.float64)
                for B in batches:
                    x32 = inputs.make_activations(B, K, inputs.activation_seed(cfg, B) + li, lognormal_channels=lognormal)
                    x = torch.from_numpy(x32).to(dev).to(torch.bfloat16)
                    t = time_product(hb, torch, stream, q, B, x, reps=100)
                    par = parity_on_sampled_rows(hb, oracle, q, x32, t["y"], xi, g64)
                    row = product_row(hb, q, B, t, peak, peak_tf, par)
                    row["workload"] = workload + (" (log-normal channel scales)" if lognormal else "")
                    rows.append(row)
                del q
        if workload == "llama-3.1-8b" and not lognormal:
            continue            # the 8B weights are used again by the next entry
        cache.clear()
    return rows


# --------------------------------------------------------------------------------------------- our arm
def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2411_17525_b200 as hb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the HIGGS kernels have no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    layers = inputs.LAYER_SETS[args.workload]
    names = [nm for nm, _, _ in layers]
    cfg = inputs.CONFIG_OF_SET[args.workload]
    pn, grid_text = layer_grids(args, layers, cfg)
    xi = inputs.rht_seed(cfg)
    B = args.batch
    peak, peak_tf, peak_src = measured_peaks()

    def ev():
        return torch.cuda.Event(enable_timing=True)

    # ---- E0: grid fit on the device (Algorithm 2), 2^18 seeded Gaussian samples (the host recipe both arms share)
    grids, grid_info = {}, {}

    def fit_grid(key):
        if key not in grids:
            p, n = key
            samples = torch.from_numpy(inputs.gaussian_samples(p, inputs.grid_sample_seed(p, n)).astype(np.float32)).to(dev)
            e0, e1 = ev(), ev()
            e0.record()
            grids[key], mse, iters = hb.higgs_make_grid(p, n, samples, max_iters=3000)
            e1.record()
            torch.cuda.synchronize()
            it = int(iters)         # negative: the iteration limit was reached before the assignment stopped changing
            grid_info[f"p={p} n={n}"] = {"ms": e0.elapsed_time(e1), "iters": abs(it), "converged": it > 0, "max_iters": 3000,
                                         "mse": float(mse)}
        return grids[key]

    for key in sorted(set(pn)):
        fit_grid(key)

    # ---- E1-E4: encode every layer once on the device (Algorithm 1)
    set_bytes = sum(layer_bytes(N, K, *pn[li]) for li, (_, N, K) in enumerate(layers))
    copies = min(64, max(2, -(-(512 << 20) // set_bytes)))      # rotating copies (>= 512 MB in all) so that no step finds its codes in L2
    qs, xs, xs_host, xs32, ws, ys = [], [], [], [], [], []
    tables = {key: hb.higgs_make_encoder_table(key[0], key[1], grids[key]) for key in set(pn)}     # once per grid
    Ws = []
    for li, (name, N, K) in enumerate(layers):
        W = torch.from_numpy(inputs.make_weights(N, K, inputs.weight_seed(cfg, li), bf16=True)).to(dev).to(torch.bfloat16)
        q = Quantized(hb, torch, dev, name, N, K, pn[li], xi, grids[pn[li]], W, table=tables[pn[li]])
        Ws.append(W)
        qs.append(q)
        # q/k/v read the same block input, so do gate/up
        xi_of = {"k": "q", "v": "q", "up": "gate"}.get(name, name)
        if xi_of != name:                  # the same pinned tensor: the block input is one buffer on the host too
            j = names.index(xi_of)
            xs_host.append(xs_host[j])
            xs32.append(xs32[j])
        else:
            xs32.append(inputs.make_activations(B, K, inputs.activation_seed(cfg, B) + names.index(xi_of)))
            xs_host.append(torch.from_numpy(xs32[-1]).to(torch.bfloat16).pin_memory())
        xs.append(xs_host[-1].to(dev))
        ws.append(torch.empty(hb.higgs_workspace_bytes(q.desc, hb.HIGGS_OP_LINEAR, B), dtype=torch.uint8, device=dev))
        ys.append(torch.empty((B, N), dtype=torch.float32, device=dev))
    descs = [q.desc for q in qs]
    # the encoder's time: one more pass over all layers into the same buffers, the calls enqueued back to back
    torch.cuda.synchronize()
    e0, e1 = ev(), ev()
    e0.record()
    for q, W in zip(qs, Ws):
        q.encode_again(hb, W)
    e1.record()
    torch.cuda.synchronize()
    enc_ms = e0.elapsed_time(e1)
    enc_weights = sum(N * K for _, N, K in layers)
    del Ws
    for q in qs:
        q.wsq = None
        q.ensure_copies(copies)

    # layers that read the same block input share one rotation (the transform is isolated from the product, Sec. 4.3);
    # a layer whose K is split across thread blocks goes through higgs_linear, whose rotation kernel also clears y
    share = {"q": "attn", "k": "attn", "v": "attn", "gate": "mlp", "up": "mlp"}
    groups_of = {}
    for li, nm in enumerate(names):
        tiled = hb.higgs_rotated_layout(descs[li], B) > 0          # tensor-core path: never split
        split = (not tiled) and hb.higgs_linear_uses_atomics(descs[li], B)
        key = (share.get(nm) + f":{hb.higgs_rotated_layout(descs[li], B)}") if (share.get(nm) and not split) else None
        groups_of.setdefault(key if key else f"own{li}", []).append(li)
    xdags = {k: torch.empty(hb.higgs_rotated_bytes(descs[v[0]], B) // 2, dtype=torch.float16, device=dev)
             for k, v in groups_of.items() if len(v) > 1}
    # a sharing group whose layers also share a grid runs as ONE product over the concatenated rows (higgs_linear_multi:
    # rows are independent); otherwise the first layer rotates for the others (higgs_linear_share)
    multis = {}
    for k, v in groups_of.items():
        if len(v) > 1 and len({qs[li].pn for li in v}) == 1:
            multis[k] = [hb.MultiLinear([descs[li] for li in v], [qs[li].packed[c] for li in v], [qs[li].scales[c] for li in v],
                                        qs[v[0]].grid, [ys[li] for li in v], B) for c in range(copies)]
    merged_names = ", ".join("|".join(names[li] for li in groups_of[k]) for k in multis) or "none"
    launches_per_step = 0
    for k, v in groups_of.items():
        if k in multis:
            launches_per_step += multis[k][0].launches
        elif len(v) > 1:    # one rotation, then one product launch per layer (per 16 tokens on the small-batch path);
                            # for 1-2 tokens the first product rotates x itself and leaves the result for the others
            first_is_one_launch = hb.higgs_linear_launch_count(descs[v[0]], B) == 1
            launches_per_step += (0 if first_is_one_launch else 1) + \
                sum(1 if hb.higgs_rotated_layout(descs[li], B) > 0 else -(-B // 16) for li in v)
        else:
            launches_per_step += hb.higgs_linear_launch_count(descs[v[0]], B)

    def step(i):
        c = i % copies
        for key, lis in groups_of.items():
            if key in multis:
                hb.higgs_linear_multi(multis[key][c], xs[lis[0]])
            elif len(lis) > 1:    # the first layer of the group also produces the rotated activations of the others
                li = lis[0]
                hb.higgs_linear_share(descs[li], xs[li], qs[li].packed[c], qs[li].scales[c], qs[li].grid, xdag_out=xdags[key],
                                      workspace=ws[li], y=ys[li])
                for li in lis[1:]:
                    hb.higgs_linear_prerotated(descs[li], xdags[key], qs[li].packed[c], qs[li].scales[c], qs[li].grid,
                                               workspace=ws[li], y=ys[li], B=B)
            else:
                li = lis[0]
                hb.higgs_linear(descs[li], xs[li], qs[li].packed[c], qs[li].scales[c], qs[li].grid, workspace=ws[li], y=ys[li])

    # end to end: one pinned host block of activations in, one pinned host block of outputs out, one library call per
    # step (higgs_linear_host_block: one copy each way, the block's products, layers with a common input and grid merged)
    x_keys = [str(id(t)) for t in xs_host]
    distinct = list({k: t for k, t in zip(x_keys, xs_host)}.items())
    host_blocks = [hb.HostBlock(descs, x_keys, distinct, [q.packed[c] for q in qs], [q.scales[c] for q in qs],
                                [q.grid for q in qs], B) for c in range(copies)]

    def step_host(i):
        hb.higgs_linear_host_block(host_blocks[i % copies])
        torch.cuda.current_stream().synchronize()   # the step's results are read on the host

    # ---- graphs of spg consecutive steps (over rotating weight copies); spg divides --steps, so exactly --steps steps
    # run from equal graphs (a graph boundary costs about 2 us on the device)
    stream = torch.cuda.Stream()
    spg = divisor_at_most(args.steps, max(1, args.steps_per_graph))
    spg_w = divisor_at_most(max(args.warmup, 3), spg)
    graphs = None
    with torch.cuda.stream(stream):
        step(0)
        stream.synchronize()
        if not args.no_graph:
            graphs = {}
            for length in {spg, spg_w}:
                graphs[length] = []
                for c in range(copies):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        for k in range(length):
                            step(c * length + k)
                    graphs[length].append(g)
            # every graph once before anything is timed: the first launch of a graph also uploads it to the device
            # (80 us for a graph of five steps), which is set-up, not a step
            for gl in graphs.values():
                for g in gl:
                    g.replay()
            stream.synchronize()

    replay_marks = []                 # (event, steps covered) after every graph replay of the last run_steps call

    def run_steps(first, count):      # exactly `count` steps, starting with step number `first`
        length = spg if count % spg == 0 else spg_w
        i = first
        replay_marks.clear()
        while count > 0:
            if graphs is not None and count >= length:
                graphs[length][(i // length) % copies].replay()
                i += length
                count -= length
                m = ev()
                m.record(stream)
                replay_marks.append((m, length))
            else:
                step(i)
                i += 1
                count -= 1

    def run_steps_host(first, count):
        for i in range(first, first + count):
            step_host(i)

    def barrier():
        if world > 1:
            dist.barrier()

    def timed(fn, steps, warmup):
        with torch.cuda.stream(stream):
            fn(0, warmup)
            stream.synchronize()
            barrier()
            torch.cuda.synchronize()
            a, b = ev(), ev()
            a.record(stream)
            fn(warmup, steps)
            b.record(stream)
            torch.cuda.synchronize()
            timed.start_event = a
            barrier()
            ms = a.elapsed_time(b)
        return max_over_ranks(ms, dev, world)

    warm = max(args.warmup, 3)
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms = timed(run_steps, args.steps, warm)
    # where the time of the timed region goes: per graph replay (the first one also carries the launch latency of the
    # first graph after the synchronisation that the protocol puts before the region)
    per_replay = None
    if replay_marks:
        prev, per = timed.start_event, []
        for m, length in replay_marks:
            per.append(prev.elapsed_time(m) * 1e3 / length)
            prev = m
        per_replay = {"us_per_step_first_replay": round(per[0], 2), "us_per_step_median": round(statistics.median(per), 2),
                      "us_per_step_min": round(min(per), 2), "replays": len(per)}
    ms_e2e = timed(run_steps_host, args.steps, warm)
    # nvidia-smi samples every 100 ms and the timed regions above last tens of milliseconds: keep the same load running
    # (untimed) for a second more so that the clock record has samples taken under it
    extra_steps = 0
    if rank == 0:
        t_probe = time.perf_counter()
        with torch.cuda.stream(stream):
            while time.perf_counter() - t_probe < 1.0:
                run_steps(extra_steps, spg)
                extra_steps += spg
                stream.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None:
        clocks["sampled_over"] = f"the timed regions and {extra_steps} more untimed steps of the same load"

    ms_per_step = ms / args.steps
    value = aggregate_value(set_bytes, args.steps, ms, world)
    e2e_value = aggregate_value(set_bytes, args.steps, ms_e2e, world)
    h2d = host_blocks[0].x_block.numel()       # the copied blocks (inputs shared by layers are there once; 256-byte padding included)
    d2h = host_blocks[0].y_block.numel()

    # ---- dominant kernel: the product kernel on the largest layer (most code bytes), timed alone with CUDA events
    import oracle
    grids64 = {k: g.cpu().numpy().astype(np.float64) for k, g in grids.items()}
    big = max(range(len(layers)), key=lambda i: qs[i].bytes)
    qb = qs[big]
    tb = time_product(hb, torch, stream, qb, B, xs[big])
    p, n = qb.pn
    alg = algorithmic_bytes(qb.N, qb.K, p, n, B)
    achieved = alg / (tb["us"] * 1e-6) / 1e9
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tpath):
        try:
            with open(tpath) as f:
                traffic = json.load(f).get(f"{args.workload}:{qb.name}:p{p}n{n}:B{B}")
        except Exception:
            traffic = None
    tiled_big = hb.higgs_rotated_layout(qb.desc, B) > 0
    kname = "linear_tc_kernel" if tiled_big else "linear_stream_kernel"
    common = {"traffic": traffic, "kernel": kname, "layer": f"{qb.name} {qb.N}x{qb.K} p={p} n={n}", "us_per_launch": tb["us"],
              "us_per_launch_median": tb["us_median"], "us_per_launch_min": tb["us_min"], "launches_timed": tb["launches"]}
    if B >= 64 and tiled_big:
        # dense-contraction regime: tensor roofline (fp16 operands; nominal fp16 peak = bf16 peak)
        tf = 2.0 * B * qb.N * qb.K / (tb["us"] * 1e-6) / 1e12
        roofline = {"bound": "tensor", "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": tf / peak_tf,
                    "peak_source": f"of {peak_src} (cuBLAS bf16 burst)", "flops": 2.0 * B * qb.N * qb.K,
                    "weight_GBps": qb.bytes / tb["us"] / 1e3, **common}
    else:
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "peak_source": f"of {peak_src}", "algorithmic_bytes": alg, "frac_of_8TBps": achieved / 8000.0, **common}
        # the secondary bound of a lookup-table kernel: every pair of weights (every weight of the 8-bit grid, every four
        # of the 2-bit grids) is one 32-lane shared-memory gather; an SM serves one such wavefront per clock
        per_lookup = {(2, 256): 2, (2, 64): 2, (1, 16): 2, (1, 8): 2, (2, 16): 4, (1, 4): 4, (1, 256): 1}[(p, n)]
        gathers = qb.N * qb.K / per_lookup / 32.0
        mhz = (clocks or {}).get("sm_mhz") or 1965.0
        gpeak = 148 * mhz * 1e6
        roofline["lut_gather"] = {"bound": "shared-memory gathers", "achieved": gathers / (tb["us"] * 1e-6) / 1e9,
                                  "peak": gpeak / 1e9, "unit": "G wavefronts/s", "frac": gathers / (tb["us"] * 1e-6) / gpeak,
                                  "note": "table lookups alone, 32 per wavefront, against 148 SMs x one wavefront per clock at "
                                          "the sampled SM clock; the code words' own loads and stores share that path"}

    detail = None
    if not args.no_detail and rank == 0 and world == 1:      # (detail times more launches with collectives-free code paths: single-GPU runs only)
        detail = {"layers": []}
        # one row per distinct (shape, grid) of the headline workload at its batch - and at the configuration's other
        # batch (32 for the 70B shapes, 16 otherwise) - each with the parity of the timed output on sampled rows
        other_B = 32 if args.workload == "llama-3.1-70b" else 16
        seen = set()
        for li, q in enumerate(qs):
            if (q.N, q.K, q.pn) in seen:
                continue
            seen.add((q.N, q.K, q.pn))
            for Bk in sorted({B, other_B}):
                if Bk == B:
                    x32, xk = xs32[li], xs[li]
                else:
                    x32 = inputs.make_activations(Bk, q.K, inputs.activation_seed(cfg, Bk) + li)
                    xk = torch.from_numpy(x32).to(dev).to(torch.bfloat16)
                t = tb if (li == big and Bk == B) else time_product(hb, torch, stream, q, Bk, xk, reps=100)
                par = parity_on_sampled_rows(hb, oracle, q, x32, t["y"], xi, grids64[q.pn])
                detail["layers"].append(product_row(hb, q, Bk, t, peak, peak_tf, par))
        # the step itself, as timed (multi-matrix products, shared rotations, fused rotations): one more step, then every
        # layer's output of that step against the oracle on sampled rows
        with torch.cuda.stream(stream):
            step(0)
            stream.synchronize()
        step_par = [parity_on_sampled_rows(hb, oracle, qs[li], xs32[li], ys[li], xi, grids64[qs[li].pn]) for li in range(len(layers))]
        detail["step_parity"] = {"max_rel": float(f"{max(p[0] for p in step_par):.3g}"),
                                 "max_over_rms": float(f"{max(p[1] for p in step_par):.3g}"),
                                 "what": "outputs of one whole step (the launches that are timed) for all layers, 16 sampled rows each"}
        if detail["step_parity"]["max_rel"] > 2e-3:
            raise SystemExit(f"parity re-check failed on the step's outputs: {detail['step_parity']}")
        detail["parity_bound"] = "max |y - y^| / max |y^| <= 2e-3 on 16 sampled rows of every timed layer, fp64 oracle on the device's codes"
        worst = max(r["parity_max_rel"] for r in detail["layers"])
        if worst > 2e-3:
            raise SystemExit(f"parity re-check failed on a timed shape: {worst}")

        # launch-latency floor: chains of kernels that do nothing, launched like the product kernels
        detail["launch_floor_us"] = {
            "one_block_per_sm_544_threads_227KB": round(launch_floor(hb, torch, stream, 148, 544, 232448), 3),
            "one_small_block": round(launch_floor(hb, torch, stream, 1, 32, 0), 3)}
        # the fit T = T0 + bytes / BW over the rows of the small-batch kernel at the headline batch
        nbytes = {(f"{q.N}x{q.K}", f"p={q.pn[0]} n={q.pn[1]}"): q.bytes for q in qs}
        pts = [(r["us"], nbytes[(r["shape"], r["grid"])]) for r in detail["layers"]
               if r["B"] == B and r["kernel"] == "linear_stream_kernel"]
        if len(pts) >= 3:
            A = np.array([[1.0, b] for _, b in pts])
            t0, slope = np.linalg.lstsq(A, np.array([u for u, _ in pts]), rcond=None)[0]
            detail["fit"] = {"T0_us": round(float(t0), 3), "BW_GBps": round(1e-3 / float(slope), 1) if slope > 0 else None,
                             "model": "us = T0 + bytes / BW over the layers of this set at the headline batch"}

    # ---- the same block with q/k/v and gate/up stored row-concatenated (rows are independent and the packed stream is
    # ordered by row tile, so the concatenation of the packed buffers IS the packed concatenated matrix): fewer, larger
    # products per block.  Layers are merged only where they share a grid.  Reported beside the per-layer launches.
    if detail is not None and all(nm in names for nm in ("q", "k", "v", "gate", "up")):
        idx = {nm: names.index(nm) for nm in names}

        def merge(group):
            out = []
            for li in group:
                for m in out:
                    if qs[m[0]].pn == qs[li].pn:
                        m.append(li)
                        break
                else:
                    out.append([li])
            return out

        merged = merge([idx["q"], idx["k"], idx["v"]]) + [[idx["o"]]] + merge([idx["gate"], idx["up"]]) + [[idx["down"]]]
        f_q, f_packed, f_scales, f_y, f_ws, f_x = [], [], [], [], [], []
        for lis in merged:
            Nf, Kf = sum(layers[li][1] for li in lis), layers[lis[0]][2]
            d = hb.make_desc(qs[lis[0]].pn[0], qs[lis[0]].pn[1], Nf, Kf, xi)
            f_q.append((d, qs[lis[0]].grid, "|".join(names[li] for li in lis)))
            if len(lis) == 1:
                f_packed.append(qs[lis[0]].packed[:copies])
                f_scales.append(qs[lis[0]].scales[:copies])
            else:
                f_packed.append([torch.cat([qs[li].packed[c] for li in lis]) for c in range(copies)])
                f_scales.append([torch.cat([qs[li].scales[c] for li in lis]) for c in range(copies)])
            f_y.append(torch.empty((B, Nf), dtype=torch.float32, device=dev))
            f_ws.append(torch.empty(hb.higgs_workspace_bytes(d, hb.HIGGS_OP_LINEAR, B), dtype=torch.uint8, device=dev))
            f_x.append(xs[lis[0]])

        def fused_step(i):
            c = i % copies
            for j, (d, grid, _) in enumerate(f_q):
                hb.higgs_linear(d, f_x[j], f_packed[j][c], f_scales[j][c], grid, workspace=f_ws[j], y=f_y[j])

        with torch.cuda.stream(stream):
            fused_step(0)
            stream.synchronize()
            fgraphs = []
            for c in range(copies):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    for k in range(spg):
                        fused_step(c * spg + k)
                fgraphs.append(g)

        def run_fused(first, count):
            i = first
            while count >= spg:
                fgraphs[(i // spg) % copies].replay()
                i += spg
                count -= spg
            for k in range(count):
                fused_step(i + k)

        ms_f = timed(run_fused, args.steps, warm)
        # the concatenated launch computes the same rows: compare with the per-layer outputs of a plain step
        with torch.cuda.stream(stream):
            step(0)
            fused_step(0)
            stream.synchronize()
        err = 0.0
        for j, lis in enumerate(merged):
            sep = torch.cat([ys[li] for li in lis], dim=1)
            err = max(err, float((f_y[j] - sep).abs().max() / sep.abs().max()))
        detail["row_concatenated"] = {
            "ms_per_step": ms_f / args.steps, "value_GBps": aggregate_value(set_bytes, args.steps, ms_f, 1),
            "launches_per_step": sum(hb.higgs_linear_launch_count(d, B) for d, _, _ in f_q),
            "layers": [f"{nm} {d.N}x{d.K} p={d.p} n={d.n}" for d, _, nm in f_q],
            "max_rel_vs_separate_launches": err}
        # the largest concatenated product alone
        jbig = max(range(len(f_q)), key=lambda j: f_packed[j][0].numel())
        if len(merged[jbig]) > 1:
            d, grid, nm = f_q[jbig]
            qcat = Quantized.from_buffers(nm, d, grid, f_packed[jbig], f_scales[jbig])
            tcat = time_product(hb, torch, stream, qcat, B, f_x[jbig], reps=100)
            detail["row_concatenated"]["largest"] = product_row(hb, qcat, B, tcat, peak, peak_tf)
            del qcat
        del fgraphs, f_packed, f_scales

    if detail is not None:
        # free the headline workload's copies before the other configurations are encoded
        for q in qs:
            del q.packed[1:], q.scales[1:]
        host_blocks = None
        multis = None
        graphs = None
        torch.cuda.empty_cache()
        detail["other_configurations"] = other_configurations(hb, torch, oracle, dev, stream, peak, peak_tf, fit_grid)
        worst = max(r["parity_max_rel"] for r in detail["other_configurations"])
        if worst > 2e-3:
            raise SystemExit(f"parity re-check failed on a timed shape: {worst}")

    # ---- CPU baseline: the oracle as it stands on this machine's cores (rank 0, single-GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        cpu = cpu_baseline(layers, pn, cfg, xi, grids64, B)

    if rank == 0:
        wps = enc_weights / (enc_ms * 1e-3)
        line = {
            "metric": "higgs_linear_effective_weight_bandwidth", "value": value, "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": warm, "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16xf16->f32", "data": "synthetic",
            "config": {"workload": f"{args.workload} layer set ({len(layers)} matrices), grid {grid_text}, g=1024, batch {B}",
                       "global_batch": B * world, "parallelism": f"replicas x{world}",
                       "l2": f"rotating {copies} weight copies ({copies * set_bytes / 1e6:.0f} MB > 126 MB L2)",
                       "launch": "direct" if args.no_graph else f"CUDA graphs of {spg} consecutive steps over rotating weight copies ({args.steps // spg} replays timed)",
                       "step": "one transformer block, 7 matrices: layers that read the same input and share a grid (here: " + merged_names + ") run as one product over their concatenated rows (higgs_linear_multi); other sharing layers share one rotation (higgs_linear_share + higgs_linear_prerotated); a layer with its own input goes through higgs_linear; for 1-2 tokens the rotation runs inside the product kernel"},
            "us_per_layer": ms_per_step * 1e3 / len(layers),
            "per_replay": per_replay,
            "weight_bytes_per_step": set_bytes,
            "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "roofline": roofline,
            "cpu_baseline": cpu,
            "quantize": {"weights_per_s": wps, "ms": enc_ms, "weights": enc_weights,
                         "calls": f"{len(layers)} higgs_quantize_prepared calls back to back (search table built once per grid), second pass into the same buffers",
                         "grid_fit": grid_info,
                         "rooflines": encoder_rooflines(wps, pn, [N * K for _, N, K in layers], clocks, peak, peak_src)},
            "detail": detail,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


# --------------------------------------------------------------------------------------------- sharded layer set
def split_units(total_units: int, world: int, rank: int):
    """[begin, end) of `total_units` units for `rank`: contiguous, the remainder to the first ranks."""
    base, extra = divmod(total_units, world)
    begin = rank * base + min(rank, extra)
    return begin, begin + base + (1 if rank < extra else 0)


def run_sharded(args):
    """ONE layer set sharded over the ranks (strong scaling): every rank encodes and multiplies its shard of every matrix
    and the kernels' epilogues write into peer-mapped buffers of all ranks (plain stores over NVLink, one per destination, no
    library kernel on peer memory).  rows: higgs_linear_gather, every rank ends a step holding the full outputs.  k:
    higgs_linear_kshard into slot buffers, a barrier, higgs_reduce_slots.  Between a step's writes and its readers
    stands the symmetric-memory barrier of the process group, enqueued on the timed stream."""
    import torch
    import torch.distributed as dist
    import torch.distributed._symmetric_memory as symm_mem

    import paper_2411_17525_b200 as hb

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the HIGGS kernels have no CPU fallback")
    if world > 8:
        raise SystemExit("a sharded layer writes into at most 8 devices' buffers")
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", "29517")
    os.environ.setdefault("RANK", "0")
    os.environ.setdefault("WORLD_SIZE", "1")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist.init_process_group("nccl", device_id=dev)

    layers = inputs.LAYER_SETS[args.workload]
    cfg = inputs.CONFIG_OF_SET[args.workload]
    pn, grid_text = layer_grids(args, layers, cfg)
    xi = inputs.rht_seed(cfg)
    B = args.batch
    peak, peak_tf, peak_src = measured_peaks()
    grids = {}
    for key in sorted(set(pn)):
        p, n = key
        samples = torch.from_numpy(inputs.gaussian_samples(p, inputs.grid_sample_seed(p, n)).astype(np.float32)).to(dev)
        grids[key], _, _ = hb.higgs_make_grid(p, n, samples, max_iters=3000)
    set_bytes = sum(layer_bytes(N, K, *pn[li]) for li, (_, N, K) in enumerate(layers))

    shards = []      # per layer: (desc, packed, scales, x, workspace, symmetric buffer, peer tensors, extra)
    for li, (name, N, K) in enumerate(layers):
        grid = grids[pn[li]]
        if args.shard == "rows":
            mult = 128 if N % (128 * world) == 0 else 16
            r0, r1 = hb.shard_rows(N, world, rank, mult)
            Ns, Ks, seed, x_cols = r1 - r0, K, xi, (0, K)
        else:
            g0, g1 = split_units(K // G, world, rank)
            Ns, Ks, seed, x_cols = N, (g1 - g0) * G, hb.higgs_shard_seed(xi, g0 * G), (g0 * G, g1 * G)
            r0 = 0
        d = hb.make_desc(pn[li][0], pn[li][1], Ns, Ks, seed)
        if Ns == 0 or Ks == 0:
            shards.append(None)
            continue
        # the shard's weights: the recipe's distribution, drawn per (layer, rank) - the sharded run is a throughput
        # measurement, parity of sharded layers is covered by the tests
        W = torch.from_numpy(inputs.make_weights(Ns, Ks, inputs.weight_seed(cfg, li) + 100 * (rank + 1), bf16=True)).to(dev).to(torch.bfloat16)
        pk, sc, _ = hb.higgs_quantize(d, W, grid)
        del W
        x_full = inputs.make_activations(B, K, inputs.activation_seed(cfg, B) + li)
        x = torch.from_numpy(np.ascontiguousarray(x_full[:, x_cols[0]:x_cols[1]])).to(dev).to(torch.bfloat16)
        ws = torch.empty(hb.higgs_workspace_bytes(d, hb.HIGGS_OP_LINEAR, B), dtype=torch.uint8, device=dev)
        shape = (B, N) if args.shard == "rows" else (world, B, N)
        buf = symm_mem.empty(shape, dtype=torch.float32, device=dev)
        hdl = symm_mem.rendezvous(buf, group=dist.group.WORLD)
        peers = [buf if r == rank else hdl.get_buffer(r, shape, torch.float32) for r in range(world)]
        shards.append((d, pk, sc, grid, x, ws, buf, hdl, peers, r0))
    live = [s for s in shards if s is not None]
    if not live:
        raise SystemExit("this rank holds no shard")
    barrier_hdl = live[0][7]

    def step(_i):
        for d, pk, sc, grid, x, ws, buf, hdl, peers, r0 in live:
            if args.shard == "rows":
                ordered = [peers[rank]] + [peers[r] for r in range(world) if r != rank]
                hb.higgs_linear_gather(d, x, pk, sc, grid, ordered, r0, workspace=ws)
            else:
                hb.higgs_linear_kshard(d, x, pk, sc, grid, peers, rank, workspace=ws)
        barrier_hdl.barrier()                      # all shards / partials of the step written, on every rank
        if args.shard == "k":
            for d, pk, sc, grid, x, ws, buf, hdl, peers, r0 in live:
                hb.higgs_reduce_slots(buf)
            barrier_hdl.barrier()                  # nobody overwrites a slot that is still being summed

    stream = torch.cuda.Stream()
    warm = max(args.warmup, 3)
    spg = divisor_at_most(args.steps, max(1, args.steps_per_graph))
    graph = None
    with torch.cuda.stream(stream):
        for i in range(warm):
            step(i)
        stream.synchronize()
        if not args.no_graph:        # spg steps per replay: the host's launch cost leaves the timed region
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=stream):
                for k in range(spg):
                    step(k)
            graph.replay()
        stream.synchronize()
        dist.barrier()
        torch.cuda.synchronize()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        if graph is not None:
            for _ in range(args.steps // spg):
                graph.replay()
        else:
            for i in range(args.steps):
                step(i)
        b.record(stream)
        torch.cuda.synchronize()
        dist.barrier()
        ms = max_over_ranks(a.elapsed_time(b), dev, world)
    # after the last step every rank holds every rank's contribution: this rank's own part must equal the plain product
    # of its shard, and nothing may be left unwritten (the buffers were never cleared, so a NaN-filled start shows holes)
    check = 0.0
    for d, pk, sc, grid, x, ws, buf, hdl, peers, r0 in live[:2]:
        y_own = hb.higgs_linear(d, x, pk, sc, grid)
        if args.shard == "rows":
            check = max(check, float((buf[:, r0:r0 + d.N] - y_own).abs().max() / y_own.abs().max()))
        elif world == 1:
            check = max(check, float((buf[0] - y_own).abs().max() / y_own.abs().max()))
        if not bool(torch.isfinite(buf).all()):
            check = float("inf")
    check = max_over_ranks(check, dev, world)
    status = hb.higgs_device_status()
    if rank == 0:
        value = set_bytes / (ms / args.steps * 1e-3) / 1e9          # the WHOLE layer set's weights per step: strong scaling
        line = {
            "metric": "higgs_linear_effective_weight_bandwidth", "value": value, "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": warm, "ms_per_step": ms / args.steps, "higher_is_better": True,
            "scaling": "strong", "vs_baseline": None, "dtype": "f16xf16->f32", "data": "synthetic",
            "config": {"workload": f"{args.workload} layer set ({len(layers)} matrices), grid {grid_text}, g=1024, batch {B}",
                       "global_batch": B, "parallelism": f"{args.shard}-sharded x{world}",
                       "l2": "one weight copy per rank (the sharded mode measures the exchange, not the L2-cold stream)",
                       "launch": "direct" if graph is None else f"CUDA graphs of {spg} steps",
                       "step": "every matrix of the block as a sharded layer: shard product with the exchange fused into the "
                               "epilogues (peer stores), symmetric-memory barrier" + (", slot-ordered sum, barrier" if args.shard == "k" else "")},
            "weight_bytes_per_step": set_bytes, "device_status": status, "own_shard_max_rel_dev": check,
            "e2e": None, "gpu_launches": None, "clocks": None, "roofline": None, "cpu_baseline": None,
            "frac_of_measured_hbm_per_gpu": value / world / peak,
        }
        print(json.dumps(line))
    dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.shard != "none":
        run_sharded(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
