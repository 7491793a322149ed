#!/usr/bin/env python
"""Benchmark of the HIGGS quantized linear layer on B200.

One "step" = one decode pass (Appendix F: rotate activations, stream codes, table lookup, contraction, reduce)
over the seven linear layers of one Llama-shaped transformer block for one batch of synthetic activations, wired as
in the block: q, k, v read one input (rotated once), o its own, gate and up one (rotated once), down its own.  The headline value is the
effective weight bandwidth (packed codes + scales bytes of the layer set / time per step).  The encoder
(Algorithm 1) and the grid fit (Algorithm 2) run once during set-up, on the GPU, and are reported separately.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload llama-3.2-1b] [--batch 1] [--grid 2,256]
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
    ap.add_argument("--workload", default="llama-3.2-1b", choices=list(inputs.LAYER_SETS))
    ap.add_argument("--batch", type=int, default=1)
    ap.add_argument("--grid", default="2,256",
                    help="p,n for every layer, or 'mixed': 3 or 4 bits per matrix (p=2 n=64 / n=256) from the seeded assignment "
                         "averaging 3.5 bits (the Llama-3.1-70B configuration)")
    ap.add_argument("--no-graph", action="store_true", help="launch kernels directly instead of replaying CUDA graphs")
    ap.add_argument("--steps-per-graph", type=int, default=8,
                    help="consecutive steps (over rotating weight copies) captured in one CUDA graph; a remainder of --steps runs "
                         "from one-step graphs")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-detail", action="store_true", help="skip the per-layer / other-batch detail measurements")
    return ap.parse_args()


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


# The encoder is bound by instruction issue (profiles/encode_pruned_kernel_...): 3748 warp instructions per
# (row, group) task of 1024 weights for p=2 n=256 (ncu, smsp__inst_executed.sum / tasks), against a peak of
# 148 SMs x 4 schedulers x 1 warp instruction per clock at the SM clock.
ENCODER_WARP_INSTR_PER_WEIGHT = {(2, 256): 3748.0 / 1024.0}


def encoder_roofline(weights_per_s, pn, clocks):
    grids = set(pn)
    if len(grids) != 1 or next(iter(grids)) not in ENCODER_WARP_INSTR_PER_WEIGHT:
        return None
    ipw = ENCODER_WARP_INSTR_PER_WEIGHT[next(iter(grids))]
    mhz = (clocks or {}).get("sm_max_mhz") or 1965.0
    peak = 148 * 4 * mhz * 1e6 / 1e9                    # G warp instructions / s
    achieved = weights_per_s * ipw / 1e9
    return {"bound": "alu", "achieved": achieved, "peak": peak, "unit": "G warp-instr/s", "frac": achieved / peak,
            "warp_instr_per_weight": ipw,
            "note": "whole higgs_quantize calls (search, pack and table build) against the issue rate of 148 SMs x 4 schedulers"}


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
def run_reference(args):
    """The fp64 oracle (as it stands) on the host cores: the same metric on a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    from synth import grids as make_grids

    layers = inputs.LAYER_SETS[args.workload]
    cfg = inputs.CONFIG_OF_SET[args.workload]
    pn, grid_text = layer_grids(args, layers, cfg)
    xi = inputs.rht_seed(cfg)
    grids = {k: make_grids.load(*k) for k in set(pn)}
    B = args.batch
    rows = 64  # rows of every layer per step: rows are independent, so this is a plain sample of the layer set
    sample = []
    for li, (name, N, K) in enumerate(layers):
        r = min(rows, N)
        W = inputs.make_weights(r, K, inputs.weight_seed(cfg, li), bf16=True).astype(np.float64)
        q = oracle.quantize(W, G, grids[pn[li]], xi)
        sc = oracle.round_scales_fp16(q.scales).astype(np.float64)
        x = inputs.make_activations(B, K, inputs.activation_seed(cfg, B) + li).astype(np.float64)
        sample.append((q.codes, sc, x, r, K, pn[li]))
    nbytes = sum(layer_bytes(r, K, *k) for _, _, _, r, K, k in sample)

    def step():
        for codes, sc, x, r, K, k in sample:
            oracle.linear_dense(x, codes, sc, G, grids[k], xi)

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
    cfg = inputs.CONFIG_OF_SET[args.workload]
    pn, grid_text = layer_grids(args, layers, cfg)
    xi = inputs.rht_seed(cfg)
    B = args.batch

    def ev():
        return torch.cuda.Event(enable_timing=True)

    # ---- E0: grid fit on the device (Algorithm 2), 2^18 seeded Gaussian samples
    grids, grid_ms, grid_iters, grid_mse = {}, 0.0, 0, 0.0
    for (p, n) in sorted(set(pn)):
        samples = torch.from_numpy(inputs.gaussian_samples(p, inputs.grid_sample_seed(p, n)).astype(np.float32)).to(dev)
        e0, e1 = ev(), ev()
        e0.record()
        grids[(p, n)], grid_mse, grid_iters = hb.higgs_make_grid(p, n, samples, max_iters=3000)
        e1.record()
        torch.cuda.synchronize()
        grid_ms += e0.elapsed_time(e1)
        del samples

    # ---- E1-E4: encode every layer once on the device (Algorithm 1)
    set_bytes = sum(layer_bytes(N, K, *pn[li]) for li, (_, N, K) in enumerate(layers))
    copies = max(2, -(-2 * L2_BYTES // set_bytes))          # rotating copies so that no step finds its codes in L2
    copies = min(copies, 64)
    descs, packed, scales, xs, xs_host, ws, ys = [], [], [], [], [], [], []
    enc_ms, enc_weights = 0.0, 0
    for li, (name, N, K) in enumerate(layers):
        d = hb.make_desc(pn[li][0], pn[li][1], N, K, xi)
        W = torch.from_numpy(inputs.make_weights(N, K, inputs.weight_seed(cfg, li), bf16=True)).to(dev).to(torch.bfloat16)
        pk, sc, _ = hb.higgs_quantize(d, W, grids[pn[li]])       # first call: the allocator fetches the output buffers
        torch.cuda.synchronize()
        e0, e1 = ev(), ev()
        e0.record()
        pk, sc, _ = hb.higgs_quantize(d, W, grids[pn[li]])       # timed: encode + pack kernels of the whole layer
        e1.record()
        torch.cuda.synchronize()
        enc_ms += e0.elapsed_time(e1)
        enc_weights += N * K
        del W
        descs.append(d)
        packed.append([pk] + [pk.clone() for _ in range(copies - 1)])
        scales.append([sc] + [sc.clone() for _ in range(copies - 1)])
        # q/k/v read the same block input, so do gate/up
        xi_of = {"k": "q", "v": "q", "up": "gate"}.get(name, name)
        x_seed = inputs.activation_seed(cfg, B) + [nm for nm, _, _ in layers].index(xi_of)
        if xi_of != name:                  # the same pinned tensor: the block input is one buffer on the host too
            xs_host.append(xs_host[[nm for nm, _, _ in layers].index(xi_of)])
        else:
            xs_host.append(torch.from_numpy(inputs.make_activations(B, K, x_seed)).to(torch.bfloat16).pin_memory())
        xs.append(xs_host[-1].to(dev))
        ws.append(torch.empty(hb.higgs_linear_host_workspace_bytes(d, B), dtype=torch.uint8, device=dev))
        ys.append(torch.empty((B, N), dtype=torch.float32, device=dev))
    ys_host = [torch.empty((B, N), dtype=torch.float32).pin_memory() for _, N, _ in layers]

    # layers that read the same block input share one rotation (the transform is isolated from the product, Sec. 4.3);
    # a layer whose K is split across thread blocks goes through higgs_linear, whose rotation kernel also clears y
    names = [nm for nm, _, _ in layers]
    share = {"q": "attn", "k": "attn", "v": "attn", "gate": "mlp", "up": "mlp"}
    groups_of = {}
    for li, nm in enumerate(names):
        tiled = hb.higgs_rotated_layout(descs[li], B) > 0          # tensor-core path: never split
        split = (not tiled) and hb.higgs_linear_k_splits(descs[li], B) > 1
        key = (share.get(nm) + f":{hb.higgs_rotated_layout(descs[li], B)}") if (share.get(nm) and not split) else None
        groups_of.setdefault(key if key else f"own{li}", []).append(li)
    xdags = {k: torch.empty(hb.higgs_rotated_bytes(descs[v[0]], B) // 2, dtype=torch.float16, device=dev)
             for k, v in groups_of.items() if len(v) > 1}
    launches_per_step = 0
    share_first = True     # the first layer of a group goes through higgs_linear_share
    for k, v in groups_of.items():
        if len(v) > 1:      # one rotation, then one product launch per layer (per 16 tokens on the small-batch path);
                            # for 1-2 tokens the first product rotates x itself and leaves the result for the others
            first_is_one_launch = share_first and hb.higgs_linear_launch_count(descs[v[0]], B) == 1
            launches_per_step += (0 if first_is_one_launch else 1) + \
                sum(1 if hb.higgs_rotated_layout(descs[li], B) > 0 else -(-B // 16) for li in v)
        else:
            launches_per_step += hb.higgs_linear_launch_count(descs[v[0]], B)

    def step(i):
        c = i % copies
        for key, lis in groups_of.items():
            if len(lis) > 1:
                rest = lis
                if share_first:       # the first layer of the group also produces the rotated activations of the others
                    li = lis[0]
                    hb.higgs_linear_share(descs[li], xs[li], packed[li][c], scales[li][c], grids[pn[li]], xdag_out=xdags[key],
                                          workspace=ws[li], y=ys[li])
                    rest = lis[1:]
                else:
                    hb.higgs_rotate_activations(descs[lis[0]], xs[lis[0]], out=xdags[key])
                for li in rest:
                    hb.higgs_linear_prerotated(descs[li], xdags[key], packed[li][c], scales[li][c], grids[pn[li]], workspace=ws[li],
                                               y=ys[li], B=B)
            else:
                li = lis[0]
                hb.higgs_linear(descs[li], xs[li], packed[li][c], scales[li][c], grids[pn[li]], workspace=ws[li], y=ys[li])

    # end to end: host activations in, host outputs out, one library call per step (higgs_linear_host_batch)
    host_batches = [hb.HostBatch(descs, xs_host, [packed[li][c] for li in range(len(descs))],
                                 [scales[li][c] for li in range(len(descs))], [grids[pn[li]] for li in range(len(descs))],
                                 ys_host, ws) for c in range(copies)]

    def step_host(i):
        hb.higgs_linear_host_batch(host_batches[i % copies])
        torch.cuda.current_stream().synchronize()   # the step's results are read on the host

    # ---- graphs: one per weight copy, replayed in rotation
    stream = torch.cuda.Stream()
    graphs = None
    with torch.cuda.stream(stream):
        step(0)
        stream.synchronize()
        spg = max(1, args.steps_per_graph)
        graphs_multi = None
        if not args.no_graph:
            graphs = []
            for c in range(copies):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    step(c)
                graphs.append(g)
            if spg > 1:          # the same steps, spg of them per graph: a graph boundary costs about 2 us on the device
                graphs_multi = []
                for c in range(copies):
                    g = torch.cuda.CUDAGraph()
                    with torch.cuda.graph(g, stream=stream):
                        for k in range(spg):
                            step(c * spg + k)
                    graphs_multi.append(g)

    def run_steps(first, count):      # exactly `count` steps, starting with step number `first`
        i = first
        while count > 0:
            if graphs_multi is not None and count >= spg:
                graphs_multi[(i // spg) % copies].replay()
                i += spg
                count -= spg
            elif graphs is not None:
                graphs[i % copies].replay()
                i += 1
                count -= 1
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
            barrier()
            ms = a.elapsed_time(b)
        return max_over_ranks(ms, dev, world)

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    ms = timed(run_steps, args.steps, max(args.warmup, 3))
    ms_e2e = timed(run_steps_host, args.steps, max(args.warmup, 3))
    # nvidia-smi samples every 100 ms and the timed regions above last tens of milliseconds: keep the same load running
    # (untimed) for a second more so that the clock record has samples taken under it
    extra_steps = 0
    if rank == 0:
        t_probe = time.perf_counter()
        with torch.cuda.stream(stream):
            while time.perf_counter() - t_probe < 1.0:      # small batches: under a profiler every launch is slow
                run_steps(extra_steps, 8)               # keeps rotating over the weight copies like the timed steps
                extra_steps += 8
                stream.synchronize()
    clocks = sampler.stop() if rank == 0 else None
    if clocks is not None:
        clocks["sampled_over"] = f"the timed regions and {extra_steps} more untimed steps of the same load"

    ms_per_step = ms / args.steps
    value = aggregate_value(set_bytes, args.steps, ms, world)
    e2e_value = aggregate_value(set_bytes, args.steps, ms_e2e, world)
    h2d = sum(t.numel() * 2 for t in {id(t): t for t in xs_host}.values())       # layers that share their input copy it once
    d2h = sum(B * N * 4 for _, N, _ in layers)

    # ---- dominant kernel: the product kernel on the largest layer, timed alone with CUDA events
    peak, peak_tf, peak_src = measured_peaks()
    big = max(range(len(layers)), key=lambda i: layers[i][1] * layers[i][2])
    _, Nb, Kb = layers[big]
    db = descs[big]

    def kernel_time(li, d, Bk, reps=200):
        """Average duration of one launch of the product kernel (pre-rotated activations), rotating weight copies."""
        xdag = hb.higgs_rotate_activations(d, xs[li] if Bk == B else
                                           torch.from_numpy(inputs.make_activations(Bk, d.K, 1)).to(torch.bfloat16).to(dev))
        yk = torch.empty((Bk, d.N), dtype=torch.float32, device=dev)
        wk = torch.empty(hb.higgs_workspace_bytes(d, hb.HIGGS_OP_LINEAR, Bk), dtype=torch.uint8, device=dev)
        per_launch_bytes = layer_bytes(d.N, d.K, d.p, d.n)
        grid = grids[(d.p, d.n)]
        need = max(2, -(-2 * L2_BYTES // per_launch_bytes))
        pks = list(packed[li])
        scs = list(scales[li])
        while len(pks) < min(need, 64):
            pks.append(pks[0].clone())
            scs.append(scs[0].clone())
        with torch.cuda.stream(stream):
            g = torch.cuda.CUDAGraph()
            hb.higgs_linear_prerotated(d, xdag, pks[0], scs[0], grid, workspace=wk, y=yk, B=Bk)
            stream.synchronize()
            with torch.cuda.graph(g, stream=stream):
                for c in range(len(pks)):
                    hb.higgs_linear_prerotated(d, xdag, pks[c], scs[c], grid, workspace=wk, y=yk, B=Bk)
            rounds = max(1, reps // len(pks))
            for _ in range(2):
                g.replay()
            stream.synchronize()
            a, b = ev(), ev()
            a.record(stream)
            for _ in range(rounds):
                g.replay()
            b.record(stream)
            stream.synchronize()
        nodes = hb.higgs_linear_launch_count(d, Bk) - 1
        return a.elapsed_time(b) * 1e3 / (rounds * len(pks)), nodes   # microseconds per call

    us_big, nodes_big = kernel_time(big, db, B)
    p, n = pn[big]
    alg = algorithmic_bytes(Nb, Kb, p, n, B)
    achieved = alg / (us_big * 1e-6) / 1e9
    traffic = None
    tpath = os.path.join(ROOT, "profiles", "traffic.json")
    if os.path.exists(tpath):
        try:
            with open(tpath) as f:
                traffic = json.load(f).get(f"{args.workload}:{layers[big][0]}:p{p}n{n}:B{B}")
        except Exception:
            traffic = None
    tiled_big = hb.higgs_rotated_layout(db, B) > 0
    kname = "linear_tc_kernel" if tiled_big else "linear_stream_kernel"
    if B >= 64 and tiled_big:
        # dense-contraction regime: tensor roofline (fp16 operands; nominal fp16 peak = bf16 peak)
        tf = 2.0 * B * Nb * Kb / (us_big * 1e-6) / 1e12
        roofline = {"bound": "tensor", "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s", "frac": tf / peak_tf,
                    "traffic": traffic, "peak_source": f"of {peak_src} (cuBLAS bf16 burst)", "kernel": kname,
                    "layer": f"{layers[big][0]} {Nb}x{Kb}", "us_per_launch": us_big, "flops": 2.0 * B * Nb * Kb,
                    "weight_GBps": layer_bytes(Nb, Kb, p, n) / us_big / 1e3}
    else:
        roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                    "traffic": traffic, "peak_source": f"of {peak_src}", "kernel": kname,
                    "layer": f"{layers[big][0]} {Nb}x{Kb}", "us_per_launch": us_big, "algorithmic_bytes": alg,
                    "frac_of_8TBps": achieved / 8000.0}

    detail = None
    if not args.no_detail and rank == 0:
        detail = {"layers": []}
        for li, (name, N, K) in enumerate(layers):
            if any(l["shape"] == f"{N}x{K}" and l["grid"] == f"p={pn[li][0]} n={pn[li][1]}" for l in detail["layers"]):
                continue
            us, _ = kernel_time(li, descs[li], B)
            wb = layer_bytes(N, K, *pn[li])
            detail["layers"].append({"name": name, "shape": f"{N}x{K}", "grid": f"p={pn[li][0]} n={pn[li][1]}", "B": B, "us": round(us, 3),
                                     "weight_GBps": round(wb / us / 1e3, 1), "frac_of_measured": round(wb / us / 1e3 / peak, 4)})
        if B != 16:
            us16, _ = kernel_time(big, db, 16)
            wb = layer_bytes(Nb, Kb, p, n)
            detail["batch16_largest_layer"] = {"us": round(us16, 3), "weight_GBps": round(wb / us16 / 1e3, 1),
                                               "frac_of_measured": round(wb / us16 / 1e3 / peak, 4)}

    # ---- the same block with q/k/v and gate/up stored row-concatenated (rows are independent and the packed stream is
    # ordered by row tile, so the concatenation of the packed buffers IS the packed concatenated matrix): 4 products
    # and 4 rotations per block instead of 7 and 4.  Reported beside the per-layer launches, not instead of them.
    if detail is not None and all(nm in names for nm in ("q", "k", "v", "gate", "up")) and len(set(pn)) == 1:
        grid = grids[pn[0]]
        idx = {nm: names.index(nm) for nm in names}
        merged = [("qkv", [idx["q"], idx["k"], idx["v"]]), ("o", [idx["o"]]), ("gate_up", [idx["gate"], idx["up"]]),
                  ("down", [idx["down"]])]
        f_desc, f_packed, f_scales, f_y, f_ws, f_x = [], [], [], [], [], []
        for nm, lis in merged:
            Nf, Kf = sum(layers[li][1] for li in lis), layers[lis[0]][2]
            d = hb.make_desc(p, n, Nf, Kf, xi)
            f_desc.append(d)
            f_packed.append([torch.cat([packed[li][c] for li in lis]) for c in range(copies)])
            f_scales.append([torch.cat([scales[li][c] for li in lis]) for c in range(copies)])
            f_y.append(torch.empty((B, Nf), dtype=torch.float32, device=dev))
            f_ws.append(torch.empty(hb.higgs_workspace_bytes(d, hb.HIGGS_OP_LINEAR, B), dtype=torch.uint8, device=dev))
            f_x.append(xs[lis[0]])

        def fused_step(i):
            c = i % copies
            for j, d in enumerate(f_desc):
                hb.higgs_linear(d, f_x[j], f_packed[j][c], f_scales[j][c], grid, workspace=f_ws[j], y=f_y[j])

        with torch.cuda.stream(stream):
            fused_step(0)
            stream.synchronize()
            fgraphs = []
            for c in range(copies):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    fused_step(c)
                fgraphs.append(g)
        def run_fused(first, count):
            for i in range(first, first + count):
                fgraphs[i % copies].replay()

        ms_f = timed(run_fused, args.steps, max(args.warmup, 3))
        # the concatenated launch computes the same rows: compare with the per-layer outputs of the last plain step
        with torch.cuda.stream(stream):
            step(0)
            fused_step(0)
            stream.synchronize()
        qkv = torch.cat([ys[idx["q"]], ys[idx["k"]], ys[idx["v"]]], dim=1)
        err = float((f_y[0] - qkv).abs().max() / qkv.abs().max())
        detail["row_concatenated"] = {
            "ms_per_step": ms_f / args.steps, "value_GBps": aggregate_value(set_bytes, args.steps, ms_f, 1),
            "launches_per_step": sum(hb.higgs_linear_launch_count(d, B) for d in f_desc),
            "layers": [f"{nm} {d.N}x{d.K}" for (nm, _), d in zip(merged, f_desc)],
            "qkv_vs_separate_max_rel": err}
        del fgraphs, f_packed, f_scales

    # ---- CPU baseline: the oracle as it stands on this machine's cores (rank 0, single-GPU runs only)
    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        import oracle
        rows = 256
        smp = []
        for li, (name, N, K) in enumerate(layers):
            r = min(rows, N)
            W = inputs.make_weights(r, K, inputs.weight_seed(cfg, li), bf16=True).astype(np.float64)
            g64 = grids[pn[li]].cpu().numpy().astype(np.float64)
            q = oracle.quantize(W, G, g64, xi)
            smp.append((q.codes, oracle.round_scales_fp16(q.scales).astype(np.float64), xs_host[li].float().numpy().astype(np.float64), g64, r, K, pn[li]))
        nb = sum(layer_bytes(r, K, *k) for *_, r, K, k in smp)
        reps, t0 = 0, time.perf_counter()
        while reps < 3 or time.perf_counter() - t0 < 10.0:
            for codes, sc, x, g64, r, K, k in smp:
                oracle.linear_dense(x, codes, sc, G, g64, xi)
            reps += 1
            if time.perf_counter() - t0 > 30.0:
                break
        dt = (time.perf_counter() - t0) / reps
        cpu = {"value": nb / dt / 1e9, "unit": "GB/s", "cores": oracle.threads(), "kind": "oracle",
               "sample": f"{rows} rows of each of the {len(layers)} layers (rows are independent), dequantise + fp64 matmul, {reps} passes"}

    if rank == 0:
        line = {
            "metric": "higgs_linear_effective_weight_bandwidth", "value": value, "unit": "GB/s", "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f16xf16->f32", "data": "synthetic",
            "config": {"workload": f"{args.workload} layer set ({len(layers)} matrices), grid {grid_text}, g=1024, batch {B}",
                       "global_batch": B * world, "parallelism": f"replicas x{world}",
                       "l2": f"rotating {copies} weight copies ({copies * set_bytes / 1e6:.0f} MB > 126 MB L2)",
                       "launch": "direct" if graphs is None else (f"CUDA graphs of {spg} consecutive steps (rotating weight copies), remainder from one-step graphs"
                                                                  if graphs_multi is not None else "one CUDA graph per step"),
                       "step": "one transformer block: activation rotations (q/k/v and gate/up share theirs where the layout allows: the first layer of the group goes through higgs_linear_share, which for 1-2 tokens rotates inside its product kernel and leaves the result for the others; a layer with its own rotation has it fused likewise when K is not split) + 7 products"},
            "us_per_layer": ms_per_step * 1e3 / len(layers),
            "weight_bytes_per_step": set_bytes,
            "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h,
                    "ms_per_step": ms_e2e / args.steps},
            "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks,
            "roofline": roofline,
            "cpu_baseline": cpu,
            "quantize": {"weights_per_s": enc_weights / (enc_ms * 1e-3), "ms": enc_ms, "weights": enc_weights,
                         "grid_fit_ms": grid_ms, "grid_fit_iters": int(grid_iters), "grid_mse": float(grid_mse),
                         "roofline": encoder_roofline(enc_weights / (enc_ms * 1e-3), pn, clocks)},
            "detail": detail,
        }
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
