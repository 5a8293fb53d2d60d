#!/usr/bin/env python
"""Benchmark of the MXFP4 linear-layer backward path (Algorithm 3) on B200.

One "step" = dgrad + wgrad of the four linear layers of one GPT block (QKV, attention output, FC1, FC2) at the
6.7B shapes (hidden 4096, FFN 16384, 8 x 2048 tokens, g = 128): four RHT + SR quantisations and two
block-scaled FP4 GEMMs per layer.  Metric: backward GEMM TFLOP/s (4 b m n per layer) INCLUDING quantisation.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--config gpt_6p7b]

Prints one JSON line (rank 0).  Legs of the GPU arm, all in this run:
  value      K steps of mxfp4_linear_backward per layer, inputs resident in HBM, CUDA events, max over ranks;
  roofline   the same step issued as its six C-ABI calls per layer with CUDA events around every call, so
             each kernel's launch duration is measured in place; the dominant kernel (the FP4 GEMM) is
             reported against the tensor peak, the quantisers against the HBM peak;
  e2e        the same metric through mxfp4_linear_backward with HOST buffers: pinned host -> device copies
             of dY, X, W and device -> host copies of dX, dW inside the timed region;
  sustained  the same step repeated for about two seconds (the board reaches its power limit), value and clocks;
  other_configs  the 1.3B and 345M layer sets, value only;
  cpu_baseline  the CPU oracle (test infrastructure, never tuned) timed on a bounded sample (rank 0, N = 1).
With N > 1 every rank runs the same workload on its own tokens (data parallel, no collective on this path): weak
scaling, value = all ranks' FLOPs / max time.  Under torchrun the ranks come from the environment; started as a
plain `python bench.py --gpus N` the script launches the N ranks itself (one process per GPU) and rank 0 prints.
"""
import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "MXFP4 backward GEMM TFLOP/s incl. RHT+SR quantize"
UNIT = "TFLOP/s"
NOMINAL_FP4_TFLOPS = 9000.0          # dense, NVIDIA's figure; context only
BF16_TO_FP4 = 4.0                    # nominal dense ratio 9 / 2.25 PFLOP/s
QUANT_BYTES_PER_ELEM = 2.0 + 0.5 + 1.0 / 32.0   # bf16 in, E2M1 code + E8M0 scale out
# DRAM bytes moved / algorithmic bytes of the GEMM, measured once with ncu on the 16384 x 4096 x 16384 launch (242.7 MB
# read + 120.5 MB written against 312.6 MB of codes, scales and bf16 output); applied to the average launch of the step.
GEMM_TRAFFIC_OVER_ALGORITHMIC = 1.16
ROUNDINGS = {"sr": 0, "rn": 1, "sr16": 2}      # the C ABI's and the oracle's rounding selectors


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"hbm_gbs": p["hbm_gbs"], "bf16_burst": p["bf16_tflops"], "bf16_sustained": p["bf16_tflops_sustained"],
                "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


# ------------------------------------------------------------------------------------------ clock sampler
class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons for one GPU while a timed region runs."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None
        self.thread = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return
        self.thread = threading.Thread(target=self._read, daemon=True)
        self.thread.start()

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append([t.strip() for t in line.split(",")])

    def mark(self):
        """Number of samples taken so far (to tell the timed region from the legs that follow it)."""
        return len(self.rows)

    def stop(self, n_timed=None):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        sm, smax, power, reasons = [], None, [], set()
        for r in self.rows:
            if len(r) < 7:
                continue
            try:
                sm.append(float(r[0])); smax = float(r[1]); power.append(float(r[2]))
            except ValueError:
                continue
            for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), r[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        sm.sort()
        # median over samples under load (at least half of the maximum power seen)
        busy = sorted(s for s, p in zip([float(r[0]) for r in self.rows if len(r) >= 7], power) if p >= 0.5 * max(power)) if power else []
        med = busy[len(busy) // 2] if busy else (sm[len(sm) // 2] if sm else None)
        out = {"sm_mhz": med, "sm_max_mhz": smax, "power_w_max": max(power) if power else None,
               "samples": len(sm), "reasons": sorted(reasons),
               "what": "nvidia-smi samples over all GPU legs of this run; sm_mhz = median of the samples under load"}
        if n_timed:
            timed = []
            for r in self.rows[:n_timed]:
                try:
                    timed.append(float(r[0]))
                except (ValueError, IndexError):
                    pass
            timed.sort()
            if timed:
                out["timed_region"] = {"samples": len(timed), "sm_mhz_median": timed[len(timed) // 2], "sm_mhz_min": timed[0]}
        return out


# ------------------------------------------------------------------------------------------ reference arm
def oracle_sample(config: str, seed: int = 0, tokens: int = 4096, dw_sample: int = 4096, rounding: str = "sr"):
    """A bounded sample of the workload for the CPU oracle: Algorithm 3 on a `tokens`-token slab of the
    attention-output layer, dX in full and dW on up to `dw_sample` sampled rows.  Returns (fn, flops, description, threads)."""
    import numpy as np
    from oracle import ref
    from paper_2502_20586_b200 import workloads as wl
    layers, g = wl.CONFIGS[config]
    layer = [l for l in layers if l.name in ("attn_out", "single")][0]
    b_s = min(tokens, layer.b)
    rng = np.random.default_rng(seed)
    std = 1e-3 if config == "single_256x512" else 1e-4
    dY = wl.grad_like(rng, (b_s, layer.m), std)
    X = wl.activation_like(rng, (b_s, layer.n), n_outlier_channels=8)
    W = wl.weight_like(rng, (layer.m, layer.n))
    dw_rows = np.sort(rng.choice(layer.m, size=min(dw_sample, layer.m), replace=False))
    flops = 2 * b_s * layer.n * layer.m + 2 * len(dw_rows) * layer.n * b_s

    def run():
        ref.linear_backward(dY, X, W, g, ROUNDINGS[rounding], seed, dw_rows=dw_rows)

    desc = (f"Algorithm 3 (g={g}, {rounding.upper()}) on a {b_s}-token slab of the {config} {layer.name} layer (n={layer.n}, m={layer.m}): "
            f"all four operand quantisations, dX in full, dW on {len(dw_rows)} sampled rows; FLOPs = GEMM MACs x 2 actually computed")
    return run, flops, desc, ref.num_threads()


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    # each step is a quarter of the cpu_baseline sample (about 2 s), so that 40 steps still end within two minutes
    run, flops, desc, cores = oracle_sample(args.config, tokens=2048, dw_sample=2048, rounding=args.rounding)
    for _ in range(min(args.warmup, 1)):
        run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        run()
    dt = (time.perf_counter() - t0) / args.steps
    val = flops / dt / 1e12
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": min(args.warmup, 1), "ms_per_step": dt * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": args.config, "sample": desc},
        "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------------------------------ multi-rank glue
def rank_seed(seed: int, rank: int) -> int:
    """Each rank draws its own tokens (data parallel): its input seed."""
    return seed + rank


def max_over_ranks(ms, ms_e2e, world: int, device):
    """Step times of the whole job = the slowest rank's (no collective runs inside the timed path itself)."""
    if world == 1:
        return ms, ms_e2e
    import torch
    import torch.distributed as dist
    t = torch.tensor([ms, ms_e2e or 0.0], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t[0]), (float(t[1]) if ms_e2e else None)


def aggregate_value(flops_per_rank: float, world: int, ms: float) -> float:
    """Whole-job TFLOP/s: every rank's FLOPs over the slowest rank's step time (weak scaling)."""
    return world * flops_per_rank / (ms * 1e-3) / 1e12


# ------------------------------------------------------------------------------------------------ GPU arm
def run_gpu(args):
    import torch
    import torch.distributed as dist
    from paper_2502_20586_b200 import binding as mx
    from paper_2502_20586_b200 import workloads as wl

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    peaks = load_peaks()
    layers, g = wl.CONFIGS[args.config]
    seed = 0
    out_dtype = mx.OUT_BF16
    data = []
    for layer in layers:
        dY, X, W = wl.layer_inputs_device(args.config, layer, seed=rank_seed(seed, rank), device=dev)
        dX = torch.empty((layer.b, layer.n), dtype=torch.bfloat16, device=dev)
        dW = torch.empty((layer.m, layer.n), dtype=torch.bfloat16, device=dev)
        data.append((layer, dY, X, W, dX, dW))
    ws_bytes = max(mx.mxfp4_linear_backward_workspace(l.b, l.m, l.n) for l in layers)
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    flops_step = sum(l.flops for l in layers)
    stream = torch.cuda.current_stream()

    rnd = ROUNDINGS[args.rounding]

    def step(rnd=rnd):
        for (layer, dY, X, W, dX, dW) in data:
            mx.mxfp4_linear_backward(dY, X, W, g, seed, rnd, out_dtype, dX=dX, dW=dW, workspace=ws)

    # ---- value: K steps, device-resident inputs
    sampler = ClockSampler(local_rank)
    sampler.start()
    for _ in range(args.warmup):
        step()
    barrier()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record(stream)
    for _ in range(args.steps):
        step()
    ev1.record(stream)
    barrier()
    ms = ev0.elapsed_time(ev1) / args.steps
    if mx.mxfp4_device_status() != 0:
        raise RuntimeError("a device-side wait timed out during the timed region")

    legs = set(args.legs.split(","))
    n_timed = sampler.mark()                    # samples up to here cover the warm-up and the timed steps
    kernels, calls_ms, gemm_tflops = {}, None, None
    fp4_peak = BF16_TO_FP4 * peaks["bf16_burst"]
    roof_burst, roof_leg_s = True, None
    if "roofline" in legs:
        # ---- roofline: the same step as its three launches per layer (one call that quantises the four operand views,
        # two GEMM calls), CUDA events around each.  Quantiser bytes: bf16 read + codes and scales written, per element.
        bufs = []
        for (layer, dY, X, W, dX, dW) in data:
            wsl = torch.empty(mx.mxfp4_linear_backward_workspace(layer.b, layer.m, layer.n), dtype=torch.uint8, device=dev)
            bufs.append((wsl, mx.mxfp4_quantize_operands(dY, X, W, g, seed, rnd, workspace=wsl)))
        records = []   # (kind, layer name, start event, end event, work)

        def timed(kind, name, work, fn):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fn(); b.record(stream)
            records.append((kind, name, a, b, work))

        def step_calls(record):
            for (layer, dY, X, W, dX, dW), (wsl, ops) in zip(data, bufs):
                fn = lambda dY=dY, X=X, W=W, wsl=wsl: mx.mxfp4_quantize_operands(dY, X, W, g, seed, rnd, workspace=wsl)
                if record:
                    # work = (algorithmic bytes with dL/dy read once for its two views, bytes if every view were a pass of its own)
                    views = 2 * dY.numel() + X.numel() + W.numel()
                    timed("quant", layer.name, ((dY.numel() + X.numel() + W.numel()) * 2.0 + views * (0.5 + 1.0 / 32.0), views * QUANT_BYTES_PER_ELEM), fn)
                else:
                    fn()
                for (a, bb, out, fl) in ((0, 1, dX, 2 * layer.b * layer.n * layer.m), (2, 3, dW, 2 * layer.m * layer.n * layer.b)):
                    fn = lambda a=a, bb=bb, out=out, ops=ops: mx.mxfp4_gemm(ops[a][0], ops[a][1], ops[bb][0], ops[bb][1],
                                                                             16.0 / 9.0 if rnd != 1 else 1.0, out_dtype, C_out=out)
                    if record:
                        timed("gemm", layer.name, fl, fn)
                    else:
                        fn()

        step_calls(False)
        torch.cuda.synchronize()
        k_roof = max(1, min(args.steps, 5))
        leg0, leg1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        leg0.record(stream)
        for _ in range(k_roof):
            step_calls(True)
        leg1.record(stream)
        barrier()
        roof_leg_s = leg0.elapsed_time(leg1) * 1e-3
        # a leg of well under a second is a burst measurement: the burst peak is its denominator
        roof_burst = roof_leg_s < 1.0
        fp4_peak = BF16_TO_FP4 * (peaks["bf16_burst"] if roof_burst else peaks["bf16_sustained"])
        agg = {}
        quant_per_view_bytes = 0.0
        for kind, name, a, b, work in records:
            d = agg.setdefault(kind, [0.0, 0.0, 0])
            if kind == "quant":
                quant_per_view_bytes += work[1]
                work = work[0]
            d[0] += a.elapsed_time(b) * 1e-3; d[1] += work; d[2] += 1
        # the three lines per layer: quantiser alone (GB/s, of HBM peak), GEMMs alone on the quantised operands
        # (TFLOP/s, of the FP4 peaks), and the layer end to end = 4bmn / (its three launches)
        per_layer = {}
        for kind, name, a, b, work in records:
            d = per_layer.setdefault(name, {"quant_s": 0.0, "quant_bytes": 0.0, "quant_view_bytes": 0.0, "gemm_s": 0.0, "flops": 0.0})
            t = a.elapsed_time(b) * 1e-3
            if kind == "quant":
                d["quant_s"] += t; d["quant_bytes"] += work[0]; d["quant_view_bytes"] += work[1]
            else:
                d["gemm_s"] += t; d["flops"] += work
        for name, d in per_layer.items():
            q_gbs, g_tf = d["quant_bytes"] / d["quant_s"] / 1e9, d["flops"] / d["gemm_s"] / 1e12
            per_layer[name] = {"quant_GB/s": q_gbs, "quant_frac_of_hbm_peak": q_gbs / peaks["hbm_gbs"],
                               "quant_per_view_GB/s": d["quant_view_bytes"] / d["quant_s"] / 1e9,
                               "quant_per_view_frac_of_hbm_peak": d["quant_view_bytes"] / d["quant_s"] / 1e9 / peaks["hbm_gbs"],
                               "gemm_TFLOP/s": g_tf, "gemm_frac_of_4x_bf16_burst": g_tf / (BF16_TO_FP4 * peaks["bf16_burst"]),
                               "gemm_frac_of_nominal_9pf": g_tf / NOMINAL_FP4_TFLOPS,
                               "layer_TFLOP/s": d["flops"] / (d["quant_s"] + d["gemm_s"]) / 1e12,
                               "ms": (d["quant_s"] + d["gemm_s"]) / k_roof * 1e3}
        gemm_t, gemm_fl, gemm_n = agg["gemm"]
        gemm_bytes = k_roof * sum((l.b * l.m + l.n * l.m) * 0.53125 + l.b * l.n * 2 + (l.m * l.b + l.n * l.b) * 0.53125 + l.m * l.n * 2
                                  for l in layers)
        gemm_tflops = gemm_fl / gemm_t / 1e12
        kernels = {}
        t_, by, n_ = agg["quant"]
        kernels["quant"] = {"launches": n_, "avg_ms": t_ / n_ * 1e3, "GB/s": by / t_ / 1e9,
                            "frac_of_hbm_peak": by / t_ / 1e9 / peaks["hbm_gbs"],
                            "per_view_GB/s": quant_per_view_bytes / t_ / 1e9, "per_view_frac_of_hbm_peak": quant_per_view_bytes / t_ / 1e9 / peaks["hbm_gbs"],
                            "what": ("the four operand views of a layer (dY row-wise and transposed, W and X transposed), one or two launches; GB/s = algorithmic "
                                     "bytes with dL/dy read ONCE for its two views (2 B per input element + 0.53125 B per output element) / time; per_view = the bytes "
                                     "of four separate passes (2.53125 B per view element) / time, the figure comparable with a single-view launch")}
        kernels["gemm"] = {"launches": gemm_n, "avg_ms": gemm_t / gemm_n * 1e3, "TFLOP/s": gemm_tflops,
                           "frac_of_4x_bf16_burst": gemm_tflops / (BF16_TO_FP4 * peaks["bf16_burst"]),
                           "frac_of_4x_bf16_sustained": gemm_tflops / (BF16_TO_FP4 * peaks["bf16_sustained"]),
                           "frac_of_nominal_9pf": gemm_tflops / NOMINAL_FP4_TFLOPS}
        kernels["per_layer"] = per_layer
        calls_ms = sum(v[0] for v in agg.values()) / k_roof * 1e3
    variants = {}
    if "roofline" in legs:
        # the other stochastic-rounding reading, same step, a short run
        if args.rounding in ("sr", "sr16"):
            other = "sr16" if args.rounding == "sr" else "sr"
            for _ in range(3):
                step(ROUNDINGS[other])
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            k_var = max(1, min(args.steps, 20))
            barrier()
            a.record(stream)
            for _ in range(k_var):
                step(ROUNDINGS[other])
            b.record(stream)
            barrier()
            ms_var = a.elapsed_time(b) / k_var
            variants[other] = {"ms_per_step": ms_var, "value": flops_step / (ms_var * 1e-3) / 1e12, "steps": k_var,
                               "note": "this rank's step with the other SR reading (8-bit centred dither / 16-bit dither of the hardware convert), timed right after the main steps; compare runs with --rounding for a like-for-like number"}
        # the overlapped form of the call (MXFP4_OVERLAP=1): the second product's operands are quantised on the same SMs
        # while the first product's GEMM runs (small builds of both kernels share an SM); same outputs, alternating A/B
        if g in (32, 64, 128):
            ab = {"0": [], "1": []}
            for rep in range(3):
                for ov in ("0", "1"):
                    os.environ["MXFP4_OVERLAP"] = ov
                    step()
                    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    k_var = max(1, min(args.steps, 10))
                    torch.cuda.synchronize()
                    a.record(stream)
                    for _ in range(k_var):
                        step()
                    b.record(stream)
                    torch.cuda.synchronize()
                    ab[ov].append(a.elapsed_time(b) / k_var)
            os.environ.pop("MXFP4_OVERLAP", None)
            ms_ser, ms_ovl = sorted(ab["0"])[1], sorted(ab["1"])[1]
            variants["overlapped"] = {"ms_per_step": ms_ovl, "value": flops_step / (ms_ovl * 1e-3) / 1e12, "serial_ms_per_step_same_leg": ms_ser,
                                      "steps": k_var, "note": "median of three alternating runs of the overlapped and the serial form; the default is the serial form"}
        # the E4M3 forward pass the MXFP4 backward is compatible with (Section 4.1): y = x W^T of the same four layers
        if all(l.n % 128 == 0 and l.m % 8 == 0 for l in layers):
            fwd = [(X, W, torch.empty((l.b, l.m), dtype=torch.bfloat16, device=dev),
                    torch.empty(int(mx.lib().mxfp4_linear_forward_fp8_workspace(l.b, l.n, l.m)), dtype=torch.uint8, device=dev))
                   for (l, dY, X, W, dX, dW) in data]

            def step_fwd():
                for (X, W, y, wsf) in fwd:
                    mx.mxfp4_linear_forward_fp8(X, W, out_dtype, y=y, workspace=wsf)
            step_fwd()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            k_var = max(1, min(args.steps, 10))
            barrier()
            a.record(stream)
            for _ in range(k_var):
                step_fwd()
            b.record(stream)
            barrier()
            ms_var = a.elapsed_time(b) / k_var
            variants["fp8_forward"] = {"ms_per_step": ms_var, "value": 0.5 * flops_step / (ms_var * 1e-3) / 1e12, "unit": "TFLOP/s (2 b m n per layer)",
                                       "steps": k_var, "note": "forward GEMMs of the same layers with E4M3 operands (per-tensor scales), quantisation included; not part of the backward metric"}
            del fwd
        # the fused-producer variant (dY transformed and rounded inside the GEMM kernels), a few steps: it is several times slower
        if g in (32, 64, 128) and all(l.b % 256 == 0 and l.m % 256 == 0 for l in layers):
            def step_fused():
                for (layer, dY, X, W, dX, dW) in data:
                    mx.mxfp4_linear_backward_fused(dY, X, W, g, seed, rnd, out_dtype, dX=dX, dW=dW, workspace=ws)
            step_fused()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            k_var = max(1, min(args.steps, 3))
            barrier()
            a.record(stream)
            for _ in range(k_var):
                step_fused()
            b.record(stream)
            barrier()
            ms_var = a.elapsed_time(b) / k_var
            variants["fused_producer"] = {"ms_per_step": ms_var, "value": flops_step / (ms_var * 1e-3) / 1e12, "steps": k_var,
                                          "note": "Algorithm 3 with lines 3 and 5 inside the GEMM kernels: every 128 x 128 output tile re-quantises its A panel"}

    if gemm_tflops is not None:
        # On-box ceiling of the FP4 tensor pipe (resident operands, no loads, no epilogue): ~25 ms burst, ~0.3 s sustained.
        def ceiling(mma_per_pair):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream); fl = mx.mxfp4_fp4_ceiling(mma_per_pair); b.record(stream)
            torch.cuda.synchronize()
            return fl / (a.elapsed_time(b) * 1e-3) / 1e12
        ceiling(32000)
        ceil_burst, ceil_sust = ceiling(320000), ceiling(3200000)
        kernels["fp4_ceiling"] = {"burst_TFLOP/s": ceil_burst, "sustained_TFLOP/s": ceil_sust,
                                  "gemm_frac_of_burst": gemm_tflops / ceil_burst, "gemm_frac_of_sustained": gemm_tflops / ceil_sust,
                                  "what": "back-to-back 256x256x64 pair MMAs on shared-memory-resident operands"}
    sustained = None
    if "sustained" in legs:
        # ---- the same step for about two seconds: the board settles at its power limit; value and the clocks seen
        k_sus = max(args.steps, int(2000.0 / ms) + 1)
        mark0 = sampler.mark()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        barrier()
        a.record(stream)
        for _ in range(k_sus):
            step()
        b.record(stream)
        barrier()
        ms_sus = a.elapsed_time(b) / k_sus
        sus_clk = sorted(float(r[0]) for r in sampler.rows[mark0:] if len(r) >= 7 and r[0].replace(".", "", 1).isdigit())
        sustained = {"value": flops_step / (ms_sus * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms_sus, "steps": k_sus,
                     "seconds": ms_sus * k_sus * 1e-3, "sm_mhz_median": sus_clk[len(sus_clk) // 2] if sus_clk else None,
                     "frac_of_nominal_9pf": flops_step / (ms_sus * 1e-3) / 1e12 / NOMINAL_FP4_TFLOPS,
                     "frac_of_4x_bf16_sustained": flops_step / (ms_sus * 1e-3) / 1e12 / (BF16_TO_FP4 * peaks["bf16_sustained"]),
                     "note": "this rank's step, timed over about two seconds; `value` above is the K-step number the contract asks for"}
    other_configs = {}
    if "other_configs" in legs and world == 1:
        # ---- the smaller layer sets (value only): 1.3B (g = 128) and 345M (g = 64)
        for cfg in ("gpt_1p3b", "gpt_345m"):
            if cfg == args.config:
                continue
            lay2, g2 = wl.CONFIGS[cfg]
            d2 = []
            for layer in lay2:
                dY, X, W = wl.layer_inputs_device(cfg, layer, seed=seed, device=dev)
                d2.append((layer, dY, X, W, torch.empty((layer.b, layer.n), dtype=torch.bfloat16, device=dev),
                           torch.empty((layer.m, layer.n), dtype=torch.bfloat16, device=dev)))
            ws2 = torch.empty(max(mx.mxfp4_linear_backward_workspace(l.b, l.m, l.n) for l in lay2), dtype=torch.uint8, device=dev)

            def step2():
                for (layer, dY, X, W, dX, dW) in d2:
                    mx.mxfp4_linear_backward(dY, X, W, g2, seed, rnd, out_dtype, dX=dX, dW=dW, workspace=ws2)
            for _ in range(5):
                step2()
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            torch.cuda.synchronize()
            a.record(stream)
            for _ in range(20):
                step2()
            b.record(stream)
            torch.cuda.synchronize()
            ms2 = a.elapsed_time(b) / 20
            fl2 = sum(l.flops for l in lay2)
            other_configs[cfg] = {"value": fl2 / (ms2 * 1e-3) / 1e12, "unit": UNIT, "ms_per_step": ms2, "steps": 20, "g": g2,
                                  "frac_of_nominal_9pf": fl2 / (ms2 * 1e-3) / 1e12 / NOMINAL_FP4_TFLOPS}
            # the same step captured once into a CUDA graph and replayed: these layers' kernels last 10-40 us, so the
            # host's launch work (tensor-map encoding, three or four launches per call) shows in the eager number
            try:
                gs = torch.cuda.Stream(device=dev)
                graph = torch.cuda.CUDAGraph()
                with torch.cuda.stream(gs):
                    with torch.cuda.graph(graph, stream=gs):
                        step2()
                for _ in range(5):
                    graph.replay()
                torch.cuda.synchronize()
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for _ in range(20):
                    graph.replay()
                b.record(stream)
                torch.cuda.synchronize()
                msg = a.elapsed_time(b) / 20
                other_configs[cfg]["cuda_graph"] = {"value": fl2 / (msg * 1e-3) / 1e12, "ms_per_step": msg, "steps": 20}
                del graph
            except RuntimeError as exc:                             # capture is a convenience of this leg, not part of the path
                other_configs[cfg]["cuda_graph"] = {"error": str(exc)[:200]}
            del d2, ws2
    clocks = sampler.stop(n_timed)
    ms_e2e, h2d, d2h = None, 0, 0
    if "e2e" in legs:
        # ---- e2e: host buffers, copies inside the timed region
        host = []
        h2d = d2h = 0
        for (layer, dY, X, W, dX, dW) in data:
            hin = [t.cpu().pin_memory() for t in (dY, X, W)]
            hout = [torch.empty(t.shape, dtype=t.dtype).pin_memory() for t in (dX, dW)]
            host.append((hin, hout))
            h2d += sum(t.numel() * t.element_size() for t in hin)
            d2h += sum(t.numel() * t.element_size() for t in hout)

        # Three streams: host->device copies, the library calls, device->host copies (PCIe is full duplex).  Per layer,
        # events keep a buffer from being overwritten while its previous user is still running.
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)
        ev_in = [torch.cuda.Event() for _ in data]
        ev_comp = [torch.cuda.Event() for _ in data]
        ev_out = [torch.cuda.Event() for _ in data]
        used = [False]

        def step_e2e():
            for i, ((layer, dY, X, W, dX, dW), (hin, hout)) in enumerate(zip(data, host)):
                if used[0]:
                    s_in.wait_event(ev_comp[i])                 # the previous step's call has consumed these inputs
                with torch.cuda.stream(s_in):
                    for dst, src in zip((dY, X, W), hin):
                        dst.copy_(src, non_blocking=True)
                    ev_in[i].record(s_in)
                stream.wait_event(ev_in[i])
                if used[0]:
                    stream.wait_event(ev_out[i])                # the previous step's outputs have left the device
                mx.mxfp4_linear_backward(dY, X, W, g, seed, rnd, out_dtype, dX=dX, dW=dW, workspace=ws)
                ev_comp[i].record(stream)
                s_out.wait_event(ev_comp[i])
                with torch.cuda.stream(s_out):
                    for dst, src in zip(hout, (dX, dW)):
                        dst.copy_(src, non_blocking=True)
                    ev_out[i].record(s_out)
            used[0] = True

        def join():
            for e in ev_out:
                stream.wait_event(e)

        s_in.wait_stream(stream); s_out.wait_stream(stream)
        step_e2e()
        join()
        barrier()
        k_e2e = max(1, min(args.steps, 5))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        s_in.wait_event(e0)
        for _ in range(k_e2e):
            step_e2e()
        join()
        e1.record(stream)
        barrier()
        ms_e2e = e0.elapsed_time(e1) / k_e2e

    # ---- max over ranks
    ms, ms_e2e = max_over_ranks(ms, ms_e2e, world, dev)
    value = aggregate_value(flops_step, world, ms)
    e2e_value = aggregate_value(flops_step, world, ms_e2e) if ms_e2e else None

    cpu_baseline = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline and "e2e" in legs:
        run, fl, desc, cores = oracle_sample(args.config, rounding=args.rounding)
        t0 = time.perf_counter()
        run()
        dt = time.perf_counter() - t0
        cpu_baseline = {"value": fl / dt / 1e12, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc, "seconds": dt}

    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "mxfp4", "data": "synthetic",
            "config": {"workload": args.config, "layers": {l.name: [l.b, l.n, l.m] for l in layers}, "g": g, "rounding": args.rounding.upper(),
                       "out_dtype": "bf16", "flops_per_step": flops_step, "l2": "inputs_exceed_l2",
                       "frac_of_4x_bf16_burst": value / world / (BF16_TO_FP4 * peaks["bf16_burst"]),
                       "frac_of_nominal_9pf": value / world / NOMINAL_FP4_TFLOPS, "timed_region_s": ms * args.steps * 1e-3,
                       "step_as_separate_calls_ms": calls_ms},
            "e2e": {"value": e2e_value, "unit": UNIT, "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "ms_per_step": ms_e2e},
            "gpu_launches": args.steps * sum(4 if l.b * l.m >= (1 << 25) else 3 for l in layers),   # per layer: one or two quantiser launches + two GEMMs
            "clocks": clocks,
            "roofline": None if gemm_tflops is None else {
                         "kernel": "gemm_mxf4_pair_kernel", "bound": "tensor", "achieved": gemm_tflops, "peak": fp4_peak, "unit": "TFLOP/s",
                         "frac": gemm_tflops / fp4_peak,
                         "traffic": GEMM_TRAFFIC_OVER_ALGORITHMIC * gemm_bytes / gemm_n,
                         "traffic_note": "bytes per average launch = algorithmic bytes x 1.16 (ratio from an ncu capture of the 16384x4096x16384 launch)",
                         "peak_source": (f"4 x {peaks['source']} {'burst' if roof_burst else 'sustained'} bf16 "
                                         f"({peaks['bf16_burst'] if roof_burst else peaks['bf16_sustained']} TFLOP/s; nominal dense FP4 : bf16 = 4); "
                                         f"the per-kernel leg lasted {roof_leg_s:.3f} s, so it is a "
                                         f"{'burst' if roof_burst else 'sustained'} measurement"),
                         "leg_seconds": roof_leg_s,
                         "frac_of_nominal_9pf": gemm_tflops / NOMINAL_FP4_TFLOPS,
                         "frac_of_fp4_ceiling_burst": gemm_tflops / kernels["fp4_ceiling"]["burst_TFLOP/s"],
                         "frac_of_fp4_ceiling_sustained": gemm_tflops / kernels["fp4_ceiling"]["sustained_TFLOP/s"],
                         "ceiling_note": "fp4_ceiling: this library's resident-operand pair-MMA kernel timed in this run (kernels.fp4_ceiling)"},
            "kernels": kernels,
            "variants": variants,
            "sustained": sustained,
            "other_configs": other_configs,
            "hbm_peak_gbs": peaks["hbm_gbs"], "peaks_source": peaks["source"],
            "cpu_baseline": cpu_baseline,
        }))
    if world > 1:
        dist.destroy_process_group()


def run_stub(args):
    """The multi-rank glue without a GPU: gloo ranks, a fixed step time per rank (rank r: 3 + 2 r ms), the same
    max-over-ranks reduction and whole-job aggregation as the GPU arm.  Exists for the CPU test of `--gpus N`."""
    import torch
    import torch.distributed as dist
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    if world > 1:
        dist.init_process_group("gloo")
    flops_step = 6e12
    ms_local = 3.0 + 2.0 * rank
    time.sleep(ms_local * 1e-3 * args.steps)
    ms, _ = max_over_ranks(ms_local, None, world, torch.device("cpu"))
    if rank == 0:
        print(json.dumps({"metric": METRIC, "value": aggregate_value(flops_step, world, ms), "unit": UNIT, "n_gpus": world,
                          "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak",
                          "stub": "cpu glue test: no GPU work was done", "seeds": [rank_seed(0, r) for r in range(world)]}))
    if world > 1:
        dist.destroy_process_group()


def spawn_ranks(n: int) -> int:
    """`python bench.py --gpus N` outside torchrun: start the N ranks (one process per GPU) on this node and wait."""
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        port = sock.getsockname()[1]
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={n}", "--master-addr", "127.0.0.1",
           "--master-port", str(port), os.path.abspath(__file__), *sys.argv[1:]]
    return subprocess.run(cmd).returncode


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=40)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--config", default="gpt_6p7b")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--rounding", default="sr", choices=sorted(ROUNDINGS), help="sr: 8-bit centred dither; sr16: 16-bit dither of the hardware convert; rn: Algorithm 1")
    ap.add_argument("--legs", default="value,roofline,sustained,other_configs,e2e", help="comma list of GPU legs to run (profiling runs use 'value')")
    ap.add_argument("--stub-cpu", action="store_true",
                    help="launch / aggregation glue only: gloo ranks on CPU, a fixed sleep per rank stands in for the step (used by the multi-rank CPU test)")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args.gpus))
    elif args.stub_cpu:
        run_stub(args)
    else:
        run_gpu(args)


if __name__ == "__main__":
    main()
