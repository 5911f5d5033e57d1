#!/usr/bin/env python
"""Benchmark of the layout-driven Muon hot path on B200.

One step = one pass of the whole path over the Llama-3-8B matrix set (224 matrices, 6.98 G
elements): flat bf16 gradient shards -> muon_materialize -> muon_step_batched_out (momentum,
Frobenius norm, 5 Newton-Schulz steps in bf16/fp32-accumulate on the tensor cores, fused update)
-> muon_scatter of the bf16 updates into flat shards.  Prints ONE JSON line (rank 0).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

With N > 1 (launched through torch.distributed.run) every rank runs an independent replica of the
step on its own GPU (the path has no data-path collective); the timed region is bracketed by a
barrier and the slowest rank's device time counts.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402
import torch  # noqa: E402

from paper_2609_21594_b200 import workloads as wl  # noqa: E402

LR, MU, WD = 0.02, 0.95, 0.01
METRIC = "muon_optimizer_steps_per_s"
UNIT = "steps/s"
NUM_SHARDS = 8

# DRAM bytes (read + write) of one launch of the Newton-Schulz product kernel: the mean over the three
# products (G1, G2, G3) captured with ncu on the 4096x14336 group with 3 matrices per launch
# (0.856 + 0.173 + 0.984 GB in the committed ncu summary of that kernel), scaled by 9/3 to the 9 matrices a
# benchmark launch of that group holds (matrices are independent, so traffic grows in proportion).
NS_KERNEL_DRAM_BYTES_PER_LAUNCH = (0.856e9 + 0.173e9 + 0.984e9) / 3 * (9 / 3)


# ----------------------------------------------------------------------------- helpers
def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return {"hbm_gbs": float(p["hbm_gbs"]), "bf16_burst": float(p["bf16_tflops"]),
                "bf16_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])), "source": "measured"}
    return {"hbm_gbs": 6650.0, "bf16_burst": 1590.0, "bf16_sustained": 1400.0, "source": "fallback"}


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""

    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits",
                                          "-lms", "200", "-i", str(self.index)], stdout=open(self.path, "w"),
                                         stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, power, reasons = [], [], [], set()
        try:
            with open(self.path) as f:
                for line in f:
                    parts = [p.strip() for p in line.split(",")]
                    if len(parts) < 7:
                        continue
                    try:
                        sm.append(float(parts[0]))
                        mx.append(float(parts[1]))
                        power.append(float(parts[2]))
                    except ValueError:
                        continue
                    for name, val in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), parts[3:7]):
                        if val.lower().startswith("active"):
                            reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            busy = [s for s, p in zip(sm, power) if p > 0.5 * max(power)] or sm
            out.update(sm_mhz=statistics.median(busy), sm_max_mhz=max(mx), power_w_max=max(power),
                       reasons=sorted(reasons), samples=len(sm))
        return out


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        import torch.distributed as dist

        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group(backend="nccl" if torch.cuda.is_available() else "gloo")
    return world, rank, local


def max_over_ranks(value: float, world: int, device) -> float:
    """Slowest rank's time (the step is an independent replica per rank)."""
    if world == 1:
        return value
    import torch.distributed as dist

    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist

        dist.barrier()


# ----------------------------------------------------------------------------- CPU oracle leg
def oracle_sample_seconds(shape, repeats: int = 1):
    """Times the CPU oracle (float64, as it stands) on one full Muon step of one matrix."""
    from oracle import muon_oracle as orc

    W = wl.param_np("llama8b", 0, shape).astype(np.float64)
    G = wl.bf16_bits_to_f32(wl.to_bf16_bits(wl.grad_np("llama8b", 0, 0, shape, row_scaled=True))).astype(np.float64)
    M = np.zeros(shape)
    best = float("inf")
    for _ in range(repeats):
        t0 = time.perf_counter()
        orc.muon_step(W, G, M, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC, 1e-7, True, "fp64")
        best = min(best, time.perf_counter() - t0)
    return best


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info

        return max([int(i.get("num_threads", 1)) for i in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(shapes):
    """Oracle on a bounded sample: one full Muon step on each of the two smallest distinct shapes;
    the whole-set time is extrapolated by Newton-Schulz flop count (NS is > 99 % of the oracle's time)."""
    sample = [(1024, 4096), (4096, 4096)]
    t = sum(oracle_sample_seconds(s) for s in sample)
    f_sample = wl.ns_flops(sample)[0]
    f_total = wl.ns_flops(shapes)[0]
    est = t * f_total / f_sample
    return {"value": 1.0 / est, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"one float64 Muon step on one {sample[0][0]}x{sample[0][1]} and one {sample[1][0]}x{sample[1][1]} matrix "
                      f"({t:.1f} s), extrapolated to the 224-matrix set by NS flop count (x{f_total / f_sample:.1f})"}


def run_reference(args, world, rank):
    """The reference arm: the CPU oracle as it stands, on host cores; each step is a bounded sample."""
    if rank != 0:
        return
    shapes = wl.shapes_llama8b()
    sample = (1024, 4096)
    f_ratio = wl.ns_flops(shapes)[0] / wl.ns_flops([sample])[0]
    for _ in range(args.warmup):
        oracle_sample_seconds(sample)
    times = [oracle_sample_seconds(sample) for _ in range(args.steps)]
    t = sum(times) / len(times)
    value = 1.0 / (t * f_ratio)
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama8b: 224 matrices (32 layers x {Wq, Wo 4096x4096; Wk, Wv 1024x4096; gate, up 14336x4096; down 4096x14336})",
                   "sampled": f"each step = one float64 oracle Muon step of one {sample[0]}x{sample[1]} matrix, scaled by NS flops x{f_ratio:.1f}"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": f"one {sample[0]}x{sample[1]} matrix per step, {t:.2f} s each"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- our arm
def run_ours(args, world, rank, local):
    from paper_2609_21594_b200 import binding as mb   # fails loudly when the CUDA library is missing

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Muon path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if args.config == "llama8b":
        shapes = wl.shapes_llama8b(args.layers)
    else:                                   # the other configurations: extra data points, never the headline
        shapes = wl.CONFIGS[args.config]()
    cfg, row_scaled = args.config, args.config == "llama8b"
    n_elem = sum(m * n for m, n in shapes)
    layout = wl.layout_per_param(shapes, NUM_SHARDS)
    ctx = mb.Context()
    L = mb.Layout(ctx, layout, 2)
    ctx.ensure_workspace(shapes)
    stream = torch.cuda.current_stream()

    # ---- state and inputs (seeded, synthetic; drawn on the device)
    W = [wl.device_draw(cfg, 0, i, "param", s, dev, std=0.02, dtype=torch.float32) for i, s in enumerate(shapes)]
    M = [torch.zeros(s, dtype=torch.float32, device=dev) for s in shapes]
    G = [wl.device_draw(cfg, 0, i, "grad", s, dev, std=1e-3, dtype=torch.bfloat16, row_scaled=row_scaled) for i, s in enumerate(shapes)]
    O = [torch.empty(s, dtype=torch.bfloat16, device=dev) for s in shapes]
    flat_g = torch.zeros(layout.flat_len, dtype=torch.bfloat16, device=dev)
    flat_o = torch.zeros(layout.flat_len, dtype=torch.bfloat16, device=dev)
    ctx.muon_scatter(flat_g, L, G)            # the gradients now live in the flat shard buffer
    for g in G:
        g.zero_()
    torch.cuda.synchronize()

    if args.path == "flat_state":
        # sharded-state flow: parameters and momenta live in flat fp32 shard buffers too; no whole-matrix state
        flat_w = torch.zeros(layout.flat_len, dtype=torch.float32, device=dev)
        flat_m = torch.zeros(layout.flat_len, dtype=torch.float32, device=dev)
        L4 = mb.Layout(ctx, layout, 4)
        ctx.muon_scatter(flat_w, L4, W)
        torch.cuda.synchronize()
        W, M, G, O = [], [], [], []
        torch.cuda.empty_cache()

        def one_step():
            ctx.muon_step_flat(L, flat_w, flat_g, flat_m, flat_o, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
    else:
        def one_step():
            ctx.muon_materialize(flat_g, L, G)
            ctx.muon_step_batched_out(W, G, M, O, shapes, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
            ctx.muon_scatter(flat_o, L, O)

    for _ in range(args.warmup):
        one_step()
    torch.cuda.synchronize()
    if ctx.muon_last_device_status() != 0:
        raise SystemExit("a bounded device-side wait expired during warm-up")

    # ---- device-resident timing
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)

    def timed_region():
        ctx.muon_profile_enable(True)
        ctx.muon_profile_reset()
        launches0 = ctx.muon_launch_count()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        barrier(world)
        torch.cuda.synchronize()
        e0.record(stream)
        for _ in range(args.steps):
            one_step()
        e1.record(stream)
        torch.cuda.synchronize()
        barrier(world)
        clk = sampler.stop() if rank == 0 else {}
        t = max_over_ranks(e0.elapsed_time(e1), world, dev)
        n = ctx.muon_launch_count() - launches0
        ph = ctx.muon_profile_read()
        ctx.muon_profile_enable(False)
        if ctx.muon_last_device_status() != 0:
            raise SystemExit("a bounded device-side wait expired during the timed region")
        return t, n, ph, clk

    ms, launches, phases, clocks = timed_region()
    # A region that saw a hardware or thermal slowdown, or clocks stuck low with no reason (a leftover lock), does
    # not count: measure once more.  sw_power_cap alone is normal for a dense-GEMM workload on a 1 kW part.
    bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
    stuck = 0.0
    if rank == 0 and clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
        stuck = 1.0 if (not clocks.get("reasons") and clocks["sm_mhz"] < 0.6 * clocks["sm_max_mhz"]) else 0.0
    redo = 1.0 if (rank == 0 and (bad & set(clocks.get("reasons", [])) or stuck)) else 0.0
    if max_over_ranks(redo, world, dev) > 0:
        ms, launches, phases, clocks = timed_region()
        clocks["remeasured"] = True
    ms_per_step = ms / args.steps
    value = world * 1e3 / ms_per_step

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e and args.path == "materialize":
        host_in = host_out = None
        try:
            host_in = torch.empty(layout.flat_len, dtype=torch.bfloat16).pin_memory()
            host_out = torch.empty(layout.flat_len, dtype=torch.bfloat16).pin_memory()
            pinned_ok = 1.0
        except RuntimeError:
            pinned_ok = 0.0
        # every rank must take the same branch (the timed loop contains barriers)
        if -max_over_ranks(-pinned_ok, world, dev) < 1.0:
            e2e = {"value": None, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0,
                   "error": "could not pin the host flat buffers on every rank"}
        else:
            host_in.copy_(flat_g)
            e2e_steps = max(1, min(args.steps, args.e2e_steps))
            for _ in range(2):
                ctx.muon_step_flat_host(host_in, host_out, L, W, G, M, O, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
            torch.cuda.synchronize()
            barrier(world)
            e0.record(stream)
            for _ in range(e2e_steps):
                ctx.muon_step_flat_host(host_in, host_out, L, W, G, M, O, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
            e1.record(stream)
            torch.cuda.synchronize()
            barrier(world)
            ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev) / e2e_steps
            flat_bytes = layout.flat_len * 2
            e2e = {"value": world * 1e3 / ms_e2e, "unit": UNIT, "h2d_bytes_per_step": flat_bytes, "d2h_bytes_per_step": flat_bytes,
                   "ms_per_step": ms_e2e, "steps": e2e_steps}
        del host_in, host_out

    if rank != 0:
        return
    peaks = load_peaks()
    dense, sym = wl.ns_flops(shapes)
    ns_ms, ns_launches = phases["ns"]
    ns_s_per_step = ns_ms / 1e3 / args.steps
    # The engine computes A = X X^T and A A^T on the tiles that touch the upper triangle only and mirrors
    # them, so the algorithmic work of the variant that runs is steps*(3 s^2 l + s^3) per matrix.
    achieved = sym / ns_s_per_step / 1e12
    per_launch_ms = ns_ms / max(1, ns_launches)
    roofline = {"bound": "tensor", "kernel": "ns_product_pair_kernel", "achieved": achieved, "peak": peaks["bf16_sustained"],
                "unit": "TFLOP/s", "frac": achieved / peaks["bf16_sustained"], "traffic": NS_KERNEL_DRAM_BYTES_PER_LAUNCH,
                "peak_source": f"bf16_tflops_sustained of {peaks['source']} (kernel timed inside a long step)",
                "flops_per_launch": sym / (ns_launches / args.steps), "ms_per_launch": per_launch_ms,
                "launches_per_step": ns_launches // args.steps,
                "frac_of_burst_peak": achieved / peaks["bf16_burst"], "frac_of_nominal_2250": achieved / 2250.0}
    hbm = {}
    for name, bytes_per_elem in (("momentum", 12), ("update", 12), ("gather", 4), ("scatter", 4)):
        pms, _ = phases[name]
        if pms > 0:
            gbs = n_elem * bytes_per_elem / (pms / 1e3 / args.steps) / 1e9
            hbm[name] = {"ms_per_step": pms / args.steps, "gbs": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
                         "frac_of_nominal_8000": gbs / 8000.0}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": (f"llama8b: {len(shapes)} matrices ({args.layers} layers x {{Wq, Wo 4096x4096; Wk, Wv 1024x4096; "
                                "gate, up 14336x4096; down 4096x14336}), bf16 row-scaled grads in 8 flat shards, fp32 params and momenta")
                               if cfg == "llama8b" else f"{cfg}: {len(shapes)} matrices, bf16 grads in 8 flat shards, fp32 params and momenta",
                   "elements": n_elem, "ns_steps": wl.NS_STEPS, "coeffs": list(wl.QUINTIC), "lr": LR, "mu": MU, "wd": WD,
                   "l2": "inputs_exceed_l2", "parallelism": "replicas" if world > 1 else "single",
                   "path": "materialize -> step -> scatter" if args.path == "materialize" else
                           "sharded-state flow (muon_step_flat: gather and scatter fused into the elementwise kernels)"},
        "roofline": roofline,
        "ns_tflops": {"algorithmic_symmetric": achieved, "dense_equivalent_effective": dense / ns_s_per_step / 1e12},
        "phases": {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] // args.steps} for k, v in phases.items()},
        "hbm_kernels": hbm,
        "e2e": e2e,
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if world == 1 and not args.no_cpu_baseline and cfg == "llama8b":
        line["cpu_baseline"] = cpu_baseline(shapes)
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=8)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--layers", type=int, default=32, help="layers of the Llama-3-8B set (32 = the benchmark workload)")
    ap.add_argument("--config", choices=sorted(wl.CONFIGS), default="llama8b",
                    help="llama8b is the benchmark workload; the others are extra data points")
    ap.add_argument("--path", choices=["materialize", "flat_state"], default="materialize",
                    help="materialize: the benchmark step (gather, step, scatter); flat_state: the fused sharded-state flow")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":       # host-only arm: rank 0 works, the others leave at once
        run_reference(args, int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")))
        return
    world, rank, local = dist_setup(args.gpus)
    try:
        run_ours(args, world, rank, local)
    finally:
        if world > 1:
            import torch.distributed as dist

            if dist.is_initialized():
                dist.destroy_process_group()


if __name__ == "__main__":
    main()
