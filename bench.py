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

# DRAM bytes (read + write) per launch of the Newton-Schulz product kernel, from ncu captures of the same command
# line; keyed by (config, layers).  Filled in from the committed summaries under profiles/.
NS_TRAFFIC = {("llama8b", 32): 1.767e9}
# the same capture by product (70 launches each): A = X X^T, P = aI + bA + cA A^T, X' = P X; algorithmic 1.21e9 / 0.41e9 / 2.20e9
NS_TRAFFIC_BY_PRODUCT = {("llama8b", 32): {"G1": 2.510e9, "G2": 0.384e9, "G3": 2.408e9}}
NS_TRAFFIC_NOTE = ("mean of dram__bytes_read.sum + dram__bytes_write.sum over the 210 product launches of one full-size step "
                   "(one-pass ncu launch list of this command line, summarised under profiles/); algorithmic bytes per launch: 1.27e9")


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
# Both arms estimate the whole-set oracle time the same way: one float64 Muon step of one matrix per core-size
# class (s = 1024: the 1024 x 4096 group; s = 4096: one 4096 x 4096 matrix standing for the 4096 x 4096 and
# 14336 x 4096 groups), each class scaled by its Newton-Schulz flop count (NS is > 99 % of the oracle's time).
ORACLE_SAMPLES = [(1024, 4096), (4096, 4096)]


def oracle_sample_seconds(shape):
    """Times the CPU oracle (float64, as it stands) on one full Muon step of one matrix."""
    from oracle import muon_oracle as orc

    W = wl.param_np("llama8b", 0, shape).astype(np.float64)
    G = wl.bf16_bits_to_f32(wl.to_bf16_bits(wl.grad_np("llama8b", 0, 0, shape, row_scaled=True))).astype(np.float64)
    M = np.zeros(shape)
    t0 = time.perf_counter()
    orc.muon_step(W, G, M, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC, 1e-7, True, "fp64")
    return time.perf_counter() - t0


def oracle_whole_set_seconds(shapes, t_small: float, t_big: float) -> float:
    """Whole-set estimate from the mean sample times of the two core-size classes."""
    small = [s for s in shapes if min(s) <= 1024]
    big = [s for s in shapes if min(s) > 1024]
    est = 0.0
    if small:
        est += t_small * wl.ns_flops(small)[0] / wl.ns_flops([ORACLE_SAMPLES[0]])[0]
    if big:
        est += t_big * wl.ns_flops(big)[0] / wl.ns_flops([ORACLE_SAMPLES[1]])[0]
    return est


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info

        return max([int(i.get("num_threads", 1)) for i in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def cpu_baseline(shapes, repeats: int = 3):
    """Oracle on a bounded sample (about 10 s of CPU work): `repeats` steps of each sample matrix."""
    ts = [oracle_sample_seconds(ORACLE_SAMPLES[0]) for _ in range(repeats)]
    tb = [oracle_sample_seconds(ORACLE_SAMPLES[1]) for _ in range(repeats)]
    t_small, t_big = sum(ts) / len(ts), sum(tb) / len(tb)
    est = oracle_whole_set_seconds(shapes, t_small, t_big)
    return {"value": 1.0 / est, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
            "sample": f"{repeats} float64 Muon steps each of one 1024x4096 ({t_small:.2f} s) and one 4096x4096 ({t_big:.2f} s) matrix; "
                      f"each core-size class of the 224-matrix set scaled by its NS flop count ({est:.0f} s per whole step)"}


def run_reference(args, world, rank):
    """The reference arm: the CPU oracle as it stands, on host cores.  Step j is a bounded sample -- one float64
    Muon step of the 1024 x 4096 matrix (even j) or of the 4096 x 4096 matrix (odd j) -- and the whole-set time
    is estimated exactly as the other arm's cpu_baseline does."""
    if rank != 0:
        return
    shapes = wl.shapes_llama8b()
    for j in range(args.warmup):
        oracle_sample_seconds(ORACLE_SAMPLES[j % 2])
    times = [[], []]
    for j in range(max(2, args.steps)):
        times[j % 2].append(oracle_sample_seconds(ORACLE_SAMPLES[j % 2]))
    t_small, t_big = sum(times[0]) / len(times[0]), sum(times[1]) / len(times[1])
    est = oracle_whole_set_seconds(shapes, t_small, t_big)
    value = 1.0 / est
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 / value, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": "llama8b: 224 matrices (32 layers x {Wq, Wo 4096x4096; Wk, Wv 1024x4096; gate, up 14336x4096; down 4096x14336})",
                   "sampled": "each step = one float64 oracle Muon step of one matrix (1024x4096 on even steps, 4096x4096 on odd steps); "
                              "value = 1 / (whole-set time estimated per core-size class by NS flop count)"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": f"{len(times[0])} x 1024x4096 ({t_small:.2f} s each) and {len(times[1])} x 4096x4096 ({t_big:.2f} s each)"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------- our arm
class Workload:
    """Device state of one configuration: whole matrices (materialize path) or flat shards (flat_state path)."""

    def __init__(self, mb, cfg, shapes, dev, path, layout_kind="per_param"):
        self.mb, self.cfg, self.shapes, self.path = mb, cfg, shapes, path
        self.n_elem = sum(m * n for m, n in shapes)
        row_scaled = cfg == "llama8b"
        gen = wl.layout_per_param if layout_kind == "per_param" else wl.layout_flat_concat
        # 32 equal layers in 8 shards would put every cut of the flat concatenation on a layer boundary: 7 shards there,
        # so that the cuts fall inside matrices (mid-row)
        self.layout = gen(shapes, NUM_SHARDS if layout_kind == "per_param" else NUM_SHARDS - 1)
        self.ctx = mb.Context()
        self.L = mb.Layout(self.ctx, self.layout, 2)
        self.ctx.ensure_workspace(shapes)
        ctx, L, layout = self.ctx, self.L, self.layout
        # state and inputs (seeded, synthetic; drawn on the device)
        self.W = [wl.device_draw(cfg, 0, i, "param", s, dev, std=0.02, dtype=torch.float32) for i, s in enumerate(shapes)]
        self.M = [torch.zeros(s, dtype=torch.float32, device=dev) for s in shapes]
        self.G = [wl.device_draw(cfg, 0, i, "grad", s, dev, std=1e-3, dtype=torch.bfloat16, row_scaled=row_scaled)
                  for i, s in enumerate(shapes)]
        self.O = [torch.empty(s, dtype=torch.bfloat16, device=dev) for s in shapes]
        self.flat_g = torch.zeros(layout.flat_len, dtype=torch.bfloat16, device=dev)
        self.flat_o = torch.zeros(layout.flat_len, dtype=torch.bfloat16, device=dev)
        ctx.muon_scatter(self.flat_g, L, self.G)            # the gradients now live in the flat shard buffer
        for g in self.G:
            g.zero_()
        torch.cuda.synchronize()
        if path == "flat_state":
            # sharded-state flow: parameters and momenta live in flat fp32 shard buffers too; no whole-matrix state
            self.flat_w = torch.zeros(layout.flat_len, dtype=torch.float32, device=dev)
            self.flat_m = torch.zeros(layout.flat_len, dtype=torch.float32, device=dev)
            L4 = mb.Layout(ctx, layout, 4)
            ctx.muon_scatter(self.flat_w, L4, self.W)
            torch.cuda.synchronize()
            L4.close()
            self.W, self.M, self.G, self.O = [], [], [], []
            torch.cuda.empty_cache()

    def one_step(self):
        c = self.ctx
        if self.path == "flat_state":
            c.muon_step_flat(self.L, self.flat_w, self.flat_g, self.flat_m, self.flat_o, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
        elif self.path == "copy_only":
            c.muon_materialize(self.flat_g, self.L, self.G)
            c.muon_scatter(self.flat_o, self.L, self.G)
        else:
            c.muon_materialize(self.flat_g, self.L, self.G)
            c.muon_step_batched_out(self.W, self.G, self.M, self.O, self.shapes, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
            c.muon_scatter(self.flat_o, self.L, self.O)

    def close(self):
        self.L.close()
        self.ctx.close()
        self.W = self.M = self.G = self.O = []
        self.flat_g = self.flat_o = self.flat_w = self.flat_m = None
        torch.cuda.empty_cache()


def timed_region(wk, steps, world, rank, local, dev, sample_clocks=True, phase_events=True):
    """K steps between two events on the launching stream, barrier + synchronize on both sides, max over ranks.
    phase_events: the library also records an event pair around every phase of every launch set (the per-phase times)."""
    ctx = wk.ctx
    stream = torch.cuda.current_stream()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ctx.muon_profile_enable(phase_events)
    ctx.muon_profile_reset()
    launches0, enc0 = ctx.muon_launch_count(), ctx.muon_tensor_map_encodes()
    sampler = ClockSampler(local)
    if rank == 0 and sample_clocks:
        sampler.start()
    barrier(world)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(steps):
        wk.one_step()
    e1.record(stream)
    torch.cuda.synchronize()
    barrier(world)
    clk = sampler.stop() if (rank == 0 and sample_clocks) else {}
    t = max_over_ranks(e0.elapsed_time(e1), world, dev)
    n = ctx.muon_launch_count() - launches0
    enc = ctx.muon_tensor_map_encodes() - enc0
    ph = ctx.muon_profile_read()
    ctx.muon_profile_enable(False)
    if ctx.muon_synchronize_and_check() != 0:
        raise SystemExit("a bounded device-side wait expired during the timed region")
    return t, n, ph, clk, enc


def summarize(wk, ms, steps, launches, phases, encodes, peaks, world=1):
    """Per-configuration record: step time, NS rate against the tensor roofline, HBM kernels against the copy peak."""
    dense, sym = wl.ns_flops(wk.shapes)
    ns_ms, ns_launches = phases["ns"]
    rec = {"matrices": len(wk.shapes), "elements": wk.n_elem, "ms_per_step": ms / steps, "steps_per_s": world * 1e3 * steps / ms,
           "launches_per_step": launches // steps, "ns_launches_per_step": ns_launches // steps,
           "tensor_map_encodes_per_step": encodes / steps}
    if ns_ms > 0:
        s_per_step = ns_ms / 1e3 / steps
        ach = sym / s_per_step / 1e12
        rec["ns"] = {"ms_per_step": ns_ms / steps, "tflops_algorithmic_symmetric": ach,
                     "tflops_dense_equivalent": dense / s_per_step / 1e12,
                     "frac_of_sustained_peak": ach / peaks["bf16_sustained"], "frac_of_burst_peak": ach / peaks["bf16_burst"],
                     "frac_of_nominal_2250": ach / 2250.0}
    hbm = {}
    upd_bytes = 12 if wk.path != "copy_only" else 0
    for name, bytes_per_elem in (("momentum", 12), ("update", upd_bytes), ("gather", 4), ("scatter", 4)):
        pms, _ = phases[name]
        if pms > 0 and bytes_per_elem:
            gbs = wk.n_elem * bytes_per_elem / (pms / 1e3 / steps) / 1e9
            hbm[name] = {"ms_per_step": pms / steps, "gbs": gbs, "frac_of_hbm_peak": gbs / peaks["hbm_gbs"],
                         "frac_of_nominal_8000": gbs / 8000.0}
    rec["hbm_kernels"] = hbm
    return rec


def side_config(mb, name, cfg, shapes, dev, path, steps, peaks, local, layout_kind="per_param"):
    """One of the other configurations, measured after the headline (rank 0's own GPU only, a few steps)."""
    wk = Workload(mb, cfg, shapes, dev, path, layout_kind)
    for _ in range(3):
        wk.one_step()
    torch.cuda.synchronize()
    ms, launches, phases, _, enc = timed_region(wk, steps, 1, 0, local, dev, sample_clocks=False)
    rec = summarize(wk, ms, steps, launches, phases, enc, peaks)
    if ms / steps < 1.0:
        # a step of a few hundred microseconds: the ten phase events per step are a measurable share of it, so the
        # step time comes from a second loop without them (the phase split above keeps them)
        ms2, _, _, _, _ = timed_region(wk, steps, 1, 0, local, dev, sample_clocks=False, phase_events=False)
        rec["ms_per_step_with_phase_events"] = rec["ms_per_step"]
        rec["ms_per_step"] = ms2 / steps
        rec["steps_per_s"] = 1e3 * steps / ms2
    rec["workload"] = name
    rec["steps"] = steps
    wk.close()
    return rec


def run_owner(args, world, rank, local):
    """--parallelism owner: ONE optimizer step of the whole matrix set spread over the ranks (the owner-sharded
    step of Section 6.4 / Algorithm 2): every rank holds one row shard of every parameter, momentum and gradient,
    the staged shards are all-gathered per batch, each matrix is orthogonalised by its compute owner only, updates
    are broadcast and every rank applies its slice.  Total work is fixed as N grows (strong scaling)."""
    from paper_2609_21594_b200 import binding as mb
    from paper_2609_21594_b200 import owner_sharded as osd

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Muon path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    shapes = wl.shapes_llama8b(args.layers) if args.config == "llama8b" else wl.CONFIGS[args.config]()
    ctx = mb.Context()
    comm = osd.TorchComm() if world > 1 else osd.SingleComm()
    st = osd.OwnerShardedStep(shapes, osd.CudaOps(ctx, device=dev), comm, batch_elems=args.batch_elems)
    gen = torch.Generator(device=dev)
    gen.manual_seed(wl.stream_seed(args.config, 0, rank, "owner"))
    for b in range(len(st.batches)):
        st.params[b].normal_(0.0, 0.02, generator=gen)
        st.momenta[b].zero_()
        st.grads[b].copy_(torch.randn(st.grads[b].shape, generator=gen, device=dev, dtype=torch.float32).mul_(1e-3))
    stream = torch.cuda.current_stream()
    for _ in range(args.warmup):
        st.step(LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    launches0 = ctx.muon_launch_count()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    barrier(world)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(args.steps):
        st.step(LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
    e1.record(stream)
    torch.cuda.synchronize()
    barrier(world)
    clocks = sampler.stop() if rank == 0 else {}
    ms = max_over_ranks(e0.elapsed_time(e1), world, dev) / args.steps
    launches = ctx.muon_launch_count() - launches0
    if ctx.muon_synchronize_and_check() != 0:
        raise SystemExit("a bounded device-side wait expired during the timed region")
    if rank != 0:
        return
    owned = [s for s, o in zip(shapes, st.owner_of) if o == rank]
    line = {
        "metric": METRIC, "value": 1e3 / ms, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms, "higher_is_better": True, "scaling": "strong", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": f"{args.config}: {len(shapes)} matrices row-sharded over {world} rank(s), bf16 N(0, 1e-3) grads, fp32 params and momenta",
                   "parallelism": f"owner-sharded x{world}", "batches": len(st.batches), "matrices_owned_by_rank0": len(owned),
                   "ns_steps": wl.NS_STEPS, "coeffs": list(wl.QUINTIC), "lr": LR, "mu": MU, "wd": WD, "l2": "inputs_exceed_l2"},
        "e2e": None, "gpu_launches": int(launches), "clocks": clocks,
    }
    print(json.dumps(line), flush=True)


def run_ours(args, world, rank, local):
    from paper_2609_21594_b200 import binding as mb   # fails loudly when the CUDA library is missing

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the Muon path has no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if args.config == "llama8b":
        shapes = wl.shapes_llama8b(args.layers)
    elif args.config == "moe" and args.experts:   # a cut-down MoE set for profiler captures
        shapes = wl.shapes_moe(1, args.experts)
    else:                                   # the other configurations: extra data points, never the headline
        shapes = wl.CONFIGS[args.config]()
    cfg = args.config
    peaks = load_peaks()
    wk = Workload(mb, cfg, shapes, dev, args.path, args.layout)
    ctx, layout, L = wk.ctx, wk.layout, wk.L
    stream = torch.cuda.current_stream()

    for _ in range(args.warmup):
        wk.one_step()
    torch.cuda.synchronize()
    if ctx.muon_synchronize_and_check() != 0:
        raise SystemExit("a bounded device-side wait expired during warm-up")

    # ---- device-resident timing
    ms, launches, phases, clocks, encodes = timed_region(wk, args.steps, world, rank, local, dev)
    # A region that saw a hardware or thermal slowdown, or clocks stuck low with no reason (a leftover lock), does
    # not count: measure once more.  sw_power_cap alone is normal for a dense-GEMM workload on a 1 kW part.
    bad = {"hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown"}
    stuck = 0.0
    if rank == 0 and clocks.get("sm_mhz") and clocks.get("sm_max_mhz"):
        stuck = 1.0 if (not clocks.get("reasons") and clocks["sm_mhz"] < 0.6 * clocks["sm_max_mhz"]) else 0.0
    redo = 1.0 if (rank == 0 and (bad & set(clocks.get("reasons", [])) or stuck)) else 0.0
    if max_over_ranks(redo, world, dev) > 0:
        ms, launches, phases, clocks, encodes = timed_region(wk, args.steps, world, rank, local, dev)
        clocks["remeasured"] = True
    ms_per_step = ms / args.steps
    value = world * 1e3 / ms_per_step

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e and args.path == "materialize":
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
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
            host_in.copy_(wk.flat_g)
            e2e_steps = max(1, args.e2e_steps)
            for _ in range(2):
                ctx.muon_step_flat_host(host_in, host_out, L, wk.W, wk.G, wk.M, wk.O, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
            torch.cuda.synchronize()
            barrier(world)
            e0.record(stream)
            for _ in range(e2e_steps):
                ctx.muon_step_flat_host(host_in, host_out, L, wk.W, wk.G, wk.M, wk.O, LR, MU, WD, wl.NS_STEPS, wl.QUINTIC)
            e1.record(stream)
            torch.cuda.synchronize()
            barrier(world)
            ms_e2e = max_over_ranks(e0.elapsed_time(e1), world, dev) / e2e_steps
            flat_bytes = layout.flat_len * 2
            e2e = {"value": world * 1e3 / ms_e2e, "unit": UNIT, "h2d_bytes_per_step": flat_bytes, "d2h_bytes_per_step": flat_bytes,
                   "ms_per_step": ms_e2e, "steps": e2e_steps}
        del host_in, host_out

    head = summarize(wk, ms, args.steps, launches, phases, encodes, peaks, world) if rank == 0 else None
    wk.close()

    # ---- the other configurations and the sharded-state flow, a few steps each (rank 0 reports; every rank runs
    # them so that no GPU idles while another works -- they contain no barrier)
    side = {}
    if args.side_configs and cfg == "llama8b" and args.path == "materialize" and args.layers == 32:
        side["llama8b_flat_state"] = side_config(mb, "llama8b, sharded-state flow (muon_step_flat)", "llama8b", shapes, dev,
                                                 "flat_state", 5, peaks, local)
        side["llama8b_layout_flat_concat_copy_only"] = side_config(
            mb, "llama8b, gather + scatter only, flat concatenation cut into 7 shards (cuts fall inside matrices, mid-row)", "llama8b", shapes, dev,
            "copy_only", 5, peaks, local, layout_kind="flat_concat")
        side["1b"] = side_config(mb, "1B-class stack, 112 matrices", "1b", wl.shapes_1b(), dev, "materialize", 10, peaks, local)
        side["moe"] = side_config(mb, "MoE stress, 784 matrices", "moe", wl.shapes_moe(), dev, "materialize", 5, peaks, local)
        side["tiny"] = side_config(mb, "tiny d=256 layer, 6 matrices", "tiny", wl.shapes_tiny(), dev, "materialize", 50, peaks, local)

    if rank != 0:
        return
    # Roofline of the dominant kernel (the paired tcgen05 product kernel).  The engine computes A = X X^T and A A^T
    # on every unordered pair of 128-blocks once and mirrors, so the algorithmic work of the variant that runs is
    # steps*(3 s^2 l + s^3) per matrix.
    ns = head.get("ns", {})
    ns_ms, ns_launches = phases["ns"]
    roofline = {"bound": "tensor", "kernel": "ns_product_pair_kernel", "achieved": ns.get("tflops_algorithmic_symmetric"),
                "peak": peaks["bf16_sustained"], "unit": "TFLOP/s", "frac": ns.get("frac_of_sustained_peak"),
                "traffic": NS_TRAFFIC.get((cfg, args.layers)),
                "traffic_by_product": NS_TRAFFIC_BY_PRODUCT.get((cfg, args.layers)),
                "traffic_note": NS_TRAFFIC_NOTE if NS_TRAFFIC.get((cfg, args.layers)) else "no capture for this workload",
                "peak_source": f"bf16_tflops_sustained of {peaks['source']} (kernel timed inside a long step)",
                "flops_per_launch": wl.ns_flops(shapes)[1] / max(1, ns_launches / args.steps),
                "ms_per_launch": ns_ms / max(1, ns_launches), "launches_per_step": ns_launches // args.steps,
                "frac_of_burst_peak": ns.get("frac_of_burst_peak"), "frac_of_nominal_2250": ns.get("frac_of_nominal_2250")}
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
        "data": "synthetic",
        "config": {"workload": (f"llama8b: {len(shapes)} matrices ({args.layers} layers x {{Wq, Wo 4096x4096; Wk, Wv 1024x4096; "
                                "gate, up 14336x4096; down 4096x14336}), bf16 row-scaled grads in 8 flat shards, fp32 params and momenta")
                               if cfg == "llama8b" else f"{cfg}: {len(shapes)} matrices, bf16 grads in 8 flat shards, fp32 params and momenta",
                   "elements": head["elements"], "ns_steps": wl.NS_STEPS, "coeffs": list(wl.QUINTIC), "lr": LR, "mu": MU, "wd": WD,
                   "l2": "inputs_exceed_l2", "parallelism": "replicas" if world > 1 else "single", "layout": args.layout,
                   "path": {"materialize": "materialize -> step -> scatter",
                            "flat_state": "sharded-state flow (muon_step_flat: gather and scatter fused into the elementwise kernels)",
                            "copy_only": "gather + scatter only"}[args.path]},
        "roofline": roofline,
        "ns_tflops": {"algorithmic_symmetric": ns.get("tflops_algorithmic_symmetric"),
                      "dense_equivalent_effective": ns.get("tflops_dense_equivalent")},
        "phases": {k: {"ms_per_step": v[0] / args.steps, "launches_per_step": v[1] // args.steps} for k, v in phases.items()},
        "hbm_kernels": head["hbm_kernels"],
        "tensor_map_encodes_per_step": head["tensor_map_encodes_per_step"],
        "e2e": e2e,
        "gpu_launches": int(launches),
        "clocks": clocks,
    }
    if side:
        line["configs"] = side
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
    ap.add_argument("--experts", type=int, default=0, help="with --config moe: one layer of this many experts (small profiler case)")
    ap.add_argument("--path", choices=["materialize", "flat_state", "copy_only"], default="materialize",
                    help="materialize: the benchmark step (gather, step, scatter); flat_state: the fused sharded-state flow; "
                         "copy_only: gather and scatter alone")
    ap.add_argument("--layout", choices=["per_param", "flat_concat"], default="per_param",
                    help="flat-shard layout generator: per-parameter row split, or flat concatenation cut into equal parts")
    ap.add_argument("--parallelism", choices=["replicas", "owner"], default="replicas",
                    help="replicas: every rank runs the whole step on its own copy (the benchmark); owner: one step of the "
                         "whole set spread over the ranks, each matrix orthogonalised by its compute owner")
    ap.add_argument("--batch-elems", type=int, default=1 << 31, help="with --parallelism owner: elements per gather batch")
    ap.add_argument("--e2e-steps", type=int, default=8)
    ap.add_argument("--no-side-configs", dest="side_configs", action="store_false",
                    help="skip the records of the other configurations (1B, MoE, tiny, sharded-state flow)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "ours" else args.warmup
    if args.impl == "reference":       # host-only arm: rank 0 works, the others leave at once
        run_reference(args, int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("RANK", "0")))
        return
    world, rank, local = dist_setup(args.gpus)
    try:
        if args.parallelism == "owner":
            run_owner(args, world, rank, local)
        else:
            run_ours(args, world, rank, local)
    finally:
        if world > 1:
            import torch.distributed as dist

            if dist.is_initialized():
                dist.destroy_process_group()


if __name__ == "__main__":
    main()
