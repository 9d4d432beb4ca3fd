#!/usr/bin/env python
"""Benchmark of the selective-scan hot path (forward + backward) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config I] [--impl ours|reference]

A "step" is one pass of the whole hot path over one batch of synthetic input: ssm_scan_fwd (writing the checkpoint
states) followed by ssm_scan_bwd, both through the C ABI.  The workload is the Mamba-2.8B layer shape
(batch 4, L 2048, D 5120, N 16, bf16 io, fp32 state) unless --config picks another one.  The metric is elements/s
with elements = batch * L * D.  One JSON line is printed by rank 0.

With --impl reference the fp64 CPU oracle is timed instead, as it stands, on the host cores.
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "selective-scan fwd+bwd elements/s (elements = batch*L*D); achieved HBM GB/s as % of measured B200 peak"
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes (read + write) of one launch of the dominant kernel of each direction from ncu captures at the bench
# workload itself (profiles/ssm_bwd_warp_kernel_mamba2p8b_layer.md, profiles/ssm_fwd_warp_kernel_mamba2p8b_layer.md);
# None where no capture exists.
NCU_TRAFFIC_BYTES = {3: 705.4e6 + 395.6e6}
NCU_TRAFFIC_BYTES_FWD = {3: 265.7e6 + 368.4e6}


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--config", type=int, default=3, help="index into the five synthetic workloads")
    ap.add_argument("--L", type=int, default=0, help="override the sequence length of the workload (profiling captures "
                                                     "of the long-sequence path on a shortened copy)")
    ap.add_argument("--D", type=int, default=0, help="override the channel count of the workload")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--general-A", action="store_true", help="perturb A so that no row is an arithmetic progression")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the decode-step and conv1d measurements that follow the timed region")
    return ap.parse_args()


def algorithmic_bytes(cfg):
    """Bytes the method itself must move per call (bf16/f32 io): forward reads x, delta, z, B, C and writes out;
    backward reads x, delta, z, dout, B, C and writes dx, ddelta, dz, dB, dC; A, D_skip, dA, dD once."""
    e = 2 if cfg.io == "bf16" else 4
    el = cfg.elements
    bln = cfg.batch * cfg.L * cfg.N
    small = cfg.D * cfg.N * 4 + cfg.D * 4
    fwd = 4 * e * el + 2 * e * bln + small
    bwd = 7 * e * el + 4 * e * bln + 2 * small
    return fwd, bwd


# ALU peaks of one B200 from its unit counts and clocks: 148 SMs x 128 FP32 lanes x 1.965 GHz (a multiply-add counts
# as one lane-operation) and 148 SMs x 16 special-function results per clock
FP32_LANE_OPS_PER_S = 148 * 128 * 1.965e9
MUFU_OPS_PER_S = 148 * 16 * 1.965e9


def algorithmic_alu_ops(cfg):
    """FP32 lane-operations and exponentials the method itself needs per element (batch, step, channel): forward
    4 per state (discretize 2, recurrence 1, readout 1) + 14 per element (delta * x, skip, gate, converts) and one
    exponential per state + 1 (gate); backward 13 per state (recompute 3, lambda 2, dC 1, w 2, dA 1, ddelta 1,
    lambda * B 1, dB 1, cross-channel sums 1) + 30 per element and one exponential per state + 3."""
    n = cfg.N
    return {"fwd_fp32": 4 * n + 14, "fwd_exp": n + 1, "bwd_fp32": 13 * n + 30, "bwd_exp": n + 3}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs (read-only queries)."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for ln in self.proc.stdout:
            self.lines.append(ln.strip())

    def stop(self) -> dict:
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        time.sleep(0.15)
        self.proc.terminate()
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            parts = [p.strip() for p in ln.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, v in zip(names, parts[3:7]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm)}


def max_over_ranks(value: float, device="cpu") -> float:
    """Slowest rank's value (the whole job is as slow as its slowest replica); identity for a single process."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(value)
    t = torch.tensor([value], device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_value(elements_per_rank: int, world: int, ms_per_step: float) -> float:
    """Whole-job throughput of `world` replicas that each process `elements_per_rank` per step (weak scaling)."""
    return world * elements_per_rank / (ms_per_step * 1e-3)


def kernels_per_step(plan_info: dict, bwd_plan_info: dict) -> int:
    """Kernel launches of one fwd (saving states) + bwd (given saved states) pass; each direction splits the sequence
    in time on its own terms."""
    fwd = 1 if plan_info["n_segments"] == 1 else 3        # [summary, carry,] forward
    # [adjoint pre-pass, carry (not with two segments: the pre-pass writes the inflow itself),] backward, reduction
    bwd = {1: 2, 2: 3}.get(bwd_plan_info["n_segments"], 4)
    return fwd + bwd


def workload_name(cfg) -> str:
    return (f"{cfg.name} (config {cfg.cfg_id}): batch {cfg.batch}, L {cfg.L}, D {cfg.D}, N {cfg.N}, {cfg.io} io, "
            f"fp32 state; one step = selective-scan forward (saving checkpoint states) + backward")


# ------------------------------------------------------------------------------------------------ oracle timing
def time_oracle(cfg, host, nthreads=0, batch_entries=None):
    """Times the fp64 oracle, as it stands, forward then backward, on the first `batch_entries` batch entries of the
    workload (all of them by default: every channel and every step) with `nthreads` threads (0: all cores)."""
    import numpy as np
    from oracle import ssm_oracle as O
    nb = cfg.batch if batch_entries is None else max(1, min(cfg.batch, batch_entries))
    x, dl, z, g = (np.ascontiguousarray(host[k][:nb]) for k in ("x", "delta", "z", "dout"))
    B, C = host["B"][:nb], host["C"][:nb]
    A, Dk = host["A"], host["D_skip"]
    t0 = time.perf_counter()
    O.scan_fwd(x, dl, A, B, C, D_skip=Dk, z=z, nthreads=nthreads)
    t1 = time.perf_counter()
    O.scan_bwd(x, dl, A, B, C, Dk, z, g, nthreads=nthreads)
    t2 = time.perf_counter()
    el = nb * cfg.L * cfg.D
    return {"value": el / (t2 - t0), "unit": "elements/s", "cores": nthreads if nthreads else O.threads_available(),
            "kind": "oracle",
            "sample": ("the whole workload" if nb == cfg.batch else f"batch entries 0..{nb - 1} of {cfg.batch}") +
                      f" ({el} elements), fwd {t1 - t0:.2f} s + bwd {t2 - t1:.2f} s wall",
            "fwd_elements_per_s": el / (t1 - t0)}


def cpu_baseline(cfg, host):
    """The oracle on the host cores: all cores on the whole workload, one thread on a bounded part of it (about 30
    core-seconds in total for the 2.8B layer shape; longer workloads are cut to whole batch entries / fewer steps)."""
    est_core_s = cfg.elements * cfg.N * 45e-9            # ~45 ns per state step for fwd+bwd on one core
    if est_core_s > 120:                                 # the long-sequence workload: not timed in full
        return {"skipped": f"about {est_core_s:.0f} core-seconds"}
    res = time_oracle(cfg, host, nthreads=0)
    one = time_oracle(cfg, host, nthreads=1, batch_entries=max(1, int(cfg.batch * 8.0 / est_core_s)))
    res["single_thread"] = {"value": one["value"], "unit": "elements/s", "cores": 1, "sample": one["sample"],
                            "fwd_elements_per_s": one["fwd_elements_per_s"]}
    return res


def run_reference(args, cfg):
    """The reference arm: the oracle, as it stands, on the host cores; rank 0 only."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    from paper_2312_00752_b200 import synth
    host = synth.make_inputs(cfg, seed=0)
    per_step, per_ms = [], []
    info = None
    for i in range(args.warmup + args.steps):
        t0 = time.perf_counter()
        info = time_oracle(cfg, host)          # the whole workload, all cores
        if i >= args.warmup:
            per_step.append(info["value"])
            per_ms.append((time.perf_counter() - t0) * 1e3)
        if per_step and time.perf_counter() - _T0 > 240:
            break
    v = statistics.median(per_step)
    line = {"impl": "reference", "metric": METRIC, "value": v, "unit": "elements/s", "n_gpus": args.gpus,
            "steps": len(per_step), "warmup": args.warmup, "ms_per_step": statistics.median(per_ms),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": workload_name(cfg), "batch": cfg.batch, "L": cfg.L, "D": cfg.D, "N": cfg.N,
                       "io": cfg.io, "step": "fp64 oracle forward + backward over the whole workload, all host cores"},
            "cpu_baseline": {"value": v, "unit": "elements/s", "cores": info["cores"], "kind": "oracle",
                             "sample": info["sample"]},
            "e2e": {"value": v, "unit": "elements/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))


# ------------------------------------------------------------------------------------------------ our arm
def time_shape(K, torch, dev, stream, cfg, peak, general_A=False, reps=None, zoh=False, complex_state=False,
               static_bc=False):
    """Forward (saving states) and backward times of one more workload, with timing-only inputs drawn on the device
    (same shapes and value ranges as the seeded host recipe); every repetition is timed on its own with CUDA events and
    a buffer larger than L2 is overwritten in between."""
    io_t = torch.bfloat16 if cfg.io == "bf16" else torch.float32
    g = torch.Generator(device=dev)
    g.manual_seed(1234 + cfg.cfg_id)
    shp = (cfg.batch, cfg.L, cfg.D)
    bshp = (cfg.batch, cfg.L, cfg.N, 2) if complex_state else (cfg.batch, cfg.L, cfg.N)
    rn = lambda shape: torch.randn(shape, generator=g, device=dev, dtype=torch.float32)
    t = {k: rn(shp).to(io_t) for k in ("x", "z", "dout")}
    t["B"], t["C"] = rn(bshp).to(io_t), rn(bshp).to(io_t)
    if static_bc:   # B and C as float32 parameters [D][N] (Algorithm 1)
        t["B"], t["C"] = rn((cfg.D, cfg.N)), rn((cfg.D, cfg.N))
    tau = torch.exp(torch.empty(cfg.D, device=dev).uniform_(math.log(cfg.dt_min), math.log(cfg.dt_max), generator=g))
    bias = tau + torch.log(-torch.expm1(-tau))
    t["delta"] = torch.nn.functional.softplus(0.1 * rn(shp) + bias).to(io_t)
    A = -(torch.arange(cfg.N, device=dev, dtype=torch.float32) + 1.0).repeat(cfg.D, 1)
    if general_A:
        A = A * (1.0 + 0.01 * rn((cfg.D, cfg.N)))
    if complex_state:   # S4D-Lin (Section 3.6): A_n = -1/2 + n i as (re, im) pairs
        A = torch.stack([torch.full((cfg.D, cfg.N), -0.5, device=dev),
                         torch.arange(cfg.N, device=dev, dtype=torch.float32).repeat(cfg.D, 1)], dim=-1).contiguous()
    Dk = torch.ones(cfg.D, device=dev)
    opts = dict(zoh=zoh, complex_state=complex_state) if (zoh or complex_state) else {}
    if static_bc:
        opts = dict(static_B=True, static_C=True)
    prob = K.make_problem(t["x"], t["B"], True, True, save_states=True, zoh=zoh, complex_state=complex_state,
                          static_B=static_bc, static_C=static_bc)
    out = torch.empty_like(t["x"])
    saved = torch.empty(K.saved_state_bytes(prob) // 4, dtype=torch.float32, device=dev)
    grads = {"dx": torch.empty_like(t["x"]), "ddelta": torch.empty_like(t["x"]), "dz": torch.empty_like(t["x"]),
             "dB": torch.empty_like(t["B"]), "dC": torch.empty_like(t["B"]), "dA": torch.empty_like(A),
             "dD": torch.empty_like(Dk)}
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    fwd = lambda: K.ssm_scan_fwd(t["x"], t["delta"], A, t["B"], t["C"], Dk, t["z"], save_states=True, out=out,
                                 saved_states=saved, stream=stream, general_A=general_A, **opts)
    bwd = lambda: K.ssm_scan_bwd(t["x"], t["delta"], A, t["B"], t["C"], Dk, t["z"], t["dout"], saved, outputs=grads,
                                 stream=stream, general_A=general_A, **opts)
    reps = reps or (5 if cfg.elements > 2e8 else 12)
    f_ms, b_ms = [], []
    for i in range(3 + reps):
        flush.zero_()
        e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
        e[0].record(stream); fwd(); e[1].record(stream); bwd(); e[2].record(stream)
        torch.cuda.synchronize(dev)
        if i >= 3:
            f_ms.append(e[0].elapsed_time(e[1])); b_ms.append(e[1].elapsed_time(e[2]))
    fb, bb = algorithmic_bytes(cfg)
    if complex_state:   # B, C, dB, dC are twice as wide
        esz = 2 if cfg.io == "bf16" else 4
        fb += 2 * cfg.batch * cfg.L * cfg.N * esz
        bb += 4 * cfg.batch * cfg.L * cfg.N * esz
    f, b = statistics.median(f_ms), statistics.median(b_ms)
    res = {"workload": f"config {cfg.cfg_id}: batch {cfg.batch}, L {cfg.L}, D {cfg.D}, N {cfg.N}, {cfg.io} io" +
                       (", A perturbed (no arithmetic progression: one exponential per state)" if general_A else "") +
                       (", zero-order-hold B-bar (SSM_FLAG_ZOH_BBAR)" if zoh else "") +
                       (", complex state with S4D-Lin A (SSM_FLAG_COMPLEX; plain kernels)" if complex_state else "") +
                       (", B and C as parameters (SSM_FLAG_STATIC_B | SSM_FLAG_STATIC_C)" if static_bc else ""),
           "fwd_ms": f, "bwd_ms": b, "fwd_elements_per_s": cfg.elements / (f * 1e-3),
           "bwd_elements_per_s": cfg.elements / (b * 1e-3), "step_elements_per_s": cfg.elements / ((f + b) * 1e-3),
           "fwd_frac_of_hbm_peak": fb / (f * 1e-3) / 1e9 / peak, "bwd_frac_of_hbm_peak": bb / (b * 1e-3) / 1e9 / peak,
           "plan": K.plan(prob), "bwd_plan": K.bwd_plan(prob), "repetitions": reps,
           "inputs": "drawn on the device (timing only); L2 flushed between repetitions"}
    del t, out, saved, grads, flush
    torch.cuda.empty_cache()
    return res


def run_ours(args, cfg):
    import numpy as np
    import torch
    import torch.distributed as dist
    from paper_2312_00752_b200 import binding as K, synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    K.load_library()
    io_t = torch.bfloat16 if cfg.io == "bf16" else torch.float32
    # every rank owns a batch of the same shape (weak scaling, no data-path collective); ranks differ by seed
    host = synth.make_inputs(cfg, seed=rank, perturb_A=0.01 if args.general_A else 0.0)
    pinned = {k: torch.from_numpy(v).to(io_t if k not in ("A", "D_skip") else torch.float32).pin_memory()
              for k, v in host.items()}
    NSETS = 3
    sets = []
    for _ in range(NSETS):
        sets.append({k: v.to(dev, non_blocking=True) for k, v in pinned.items()})
    d0 = sets[0]
    prob = K.make_problem(d0["x"], d0["B"], True, True, save_states=True)
    plan_info = K.plan(prob)
    bwd_plan_info = K.bwd_plan(prob)
    out = torch.empty_like(d0["x"])
    saved = torch.empty(K.saved_state_bytes(prob) // 4, dtype=torch.float32, device=dev)
    grads = {"dx": torch.empty_like(d0["x"]), "ddelta": torch.empty_like(d0["x"]), "dz": torch.empty_like(d0["x"]),
             "dB": torch.empty_like(d0["B"]), "dC": torch.empty_like(d0["B"]),
             "dA": torch.empty_like(d0["A"]), "dD": torch.empty_like(d0["D_skip"])}
    stream = torch.cuda.current_stream(dev)

    def fwd(s):
        K.ssm_scan_fwd(s["x"], s["delta"], s["A"], s["B"], s["C"], s["D_skip"], s["z"], save_states=True, out=out,
                       saved_states=saved, stream=stream)

    def bwd(s):
        K.ssm_scan_bwd(s["x"], s["delta"], s["A"], s["B"], s["C"], s["D_skip"], s["z"], s["dout"], saved,
                       outputs=grads, stream=stream)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    for i in range(max(args.warmup, 3)):
        fwd(sets[i % NSETS])
        bwd(sets[i % NSETS])
    barrier()

    # ---- device-resident timing: K steps, CUDA events on the launching stream
    ev = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(args.steps)]
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    barrier()
    t_wall = time.perf_counter()
    for i in range(args.steps):
        s = sets[i % NSETS]
        ev[i][0].record(stream)
        fwd(s)
        ev[i][1].record(stream)
        bwd(s)
        ev[i][2].record(stream)
    barrier()
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop()
    total_ms = ev[0][0].elapsed_time(ev[-1][2])
    fwd_ms = [e[0].elapsed_time(e[1]) for e in ev]
    bwd_ms = [e[1].elapsed_time(e[2]) for e in ev]
    ms_per_step = max_over_ranks(total_ms / args.steps, dev)

    # ---- end to end: pinned host inputs -> device, fwd + bwd, every result back to pinned host memory
    e2e = None
    if not args.no_e2e:
        hres = {k: torch.empty(v.shape, dtype=v.dtype).pin_memory() for k, v in {"out": out, **grads}.items()}
        names_in = ("x", "delta", "z", "dout", "B", "C", "A", "D_skip")
        h2d = sum(pinned[k].numel() * pinned[k].element_size() for k in names_in)
        d2h = sum(v.numel() * v.element_size() for v in hres.values())
        arena = torch.empty(K.host_arena_bytes(prob), dtype=torch.uint8, device=dev)

        def e2e_step():   # one library call: host buffers in, host buffers out, copies pipelined with the kernels
            K.ssm_scan_fwd_bwd_host(pinned["x"], pinned["delta"], pinned["A"], pinned["B"], pinned["C"],
                                    pinned["D_skip"], pinned["z"], pinned["dout"], device=dev, arena=arena,
                                    outputs=hres, stream=stream)

        e2e_step()
        barrier()
        n_e2e = max(3, min(args.steps, 10))
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(n_e2e):
            e2e_step()
        b.record(stream)
        barrier()
        e2e_ms = max_over_ranks(a.elapsed_time(b) / n_e2e, dev)
        e2e = {"value": job_value(cfg.elements, world, e2e_ms), "unit": "elements/s",
               "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h), "ms_per_step": e2e_ms,
               "steps": n_e2e, "api": "ssm_scan_fwd_bwd_host (pinned host buffers in and out, batch pipelined over "
                                      "copy-in / compute / copy-out streams)"}

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    fwd_bytes, bwd_bytes = algorithmic_bytes(cfg)
    peak, peak_kind = measured_peaks()
    f_ms, b_ms = statistics.mean(fwd_ms), statistics.mean(bwd_ms)
    bwd_gbs = bwd_bytes / (b_ms * 1e-3) / 1e9
    fwd_gbs = fwd_bytes / (f_ms * 1e-3) / 1e9
    alu = algorithmic_alu_ops(cfg)

    def alu_fracs(direction, ms):
        per_s = cfg.elements / (ms * 1e-3)
        return {"frac_of_fp32_lane_peak": per_s * alu[direction + "_fp32"] / FP32_LANE_OPS_PER_S,
                "frac_of_mufu_peak": per_s * alu[direction + "_exp"] / MUFU_OPS_PER_S}

    line = {
        "metric": METRIC, "value": job_value(cfg.elements, world, ms_per_step), "unit": "elements/s",
        "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms_per_step,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "io_dtype": cfg.io,
        "data": "synthetic",
        "config": {"workload": workload_name(cfg), "batch": cfg.batch, "L": cfg.L, "D": cfg.D, "N": cfg.N, "io": cfg.io,
                   "step": "ssm_scan_fwd (saving checkpoint states) + ssm_scan_bwd through the C ABI",
                   "A": "perturbed (general path)" if args.general_A else "S4D-Real -(n+1)",
                   "l2": f"inputs larger than L2 (4 x {cfg.elements * (2 if cfg.io == 'bf16' else 4) / 1e6:.0f} MB) and "
                         f"{NSETS} input sets rotated between steps",
                   "plan": plan_info, "bwd_plan": bwd_plan_info,
                   "parallelism": "replicas" if world > 1 else "single"},
        "clocks": clocks,
        "gpu_launches": kernels_per_step(plan_info, bwd_plan_info) * args.steps,
        "fwd": {"ms": f_ms, "elements_per_s": cfg.elements / (f_ms * 1e-3), "algorithmic_bytes": fwd_bytes,
                "achieved_gbs": fwd_gbs, "frac_of_hbm_peak": fwd_gbs / peak, **alu_fracs("fwd", f_ms),
                "traffic": NCU_TRAFFIC_BYTES_FWD.get(cfg.cfg_id) if not args.general_A else None},
        "bwd": {"ms": b_ms, "elements_per_s": cfg.elements / (b_ms * 1e-3), "algorithmic_bytes": bwd_bytes,
                "achieved_gbs": bwd_gbs, "frac_of_hbm_peak": bwd_gbs / peak, **alu_fracs("bwd", b_ms)},
        "roofline": {"bound": "hbm", "binding_bound": "alu (FP32 lanes; see roofline_alu)",
                     "kernel": "ssm_scan_bwd call (ssm_bwd_warp_kernel, the dominant kernel, timed together with the "
                               "adjoint pre-pass and reduction kernels of the same call)",
                     "achieved": bwd_gbs, "peak": peak, "peak_kind": f"{peak_kind} copy bandwidth",
                     "unit": "GB/s", "frac": bwd_gbs / peak,
                     "traffic": NCU_TRAFFIC_BYTES.get(cfg.cfg_id) if not args.general_A else None,
                     "algorithmic_bytes": bwd_bytes},
        # the same launch against the ALU roof that actually binds it (algorithmic FP32 lane-operations per second
        # over lanes x clock); the HBM figure above is the metric, this one says how far the kernel is from its bound
        "roofline_alu": {"bound": "alu", "kernel": "ssm_scan_bwd call",
                         "achieved": cfg.elements / (b_ms * 1e-3) * alu["bwd_fp32"] / 1e12,
                         "peak": FP32_LANE_OPS_PER_S / 1e12, "unit": "T lane-op/s (FP32, FMA = 1)",
                         "frac": alu_fracs("bwd", b_ms)["frac_of_fp32_lane_peak"],
                         "ops_per_element": alu["bwd_fp32"]},
        "wall_s_timed_region": t_wall,
    }
    # the single recurrent step (decode): one pass over the float32 state, batch 64 at the same width
    try:
        if args.no_extras:
            raise RuntimeError("skipped (--no-extras)")
        sb = 64
        hs = torch.zeros((sb, cfg.D, cfg.N), dtype=torch.float32, device=dev)
        xs = torch.randn((sb, cfg.D), device=dev).to(io_t)
        ds_ = (torch.rand((sb, cfg.D), device=dev) * 0.1).to(io_t)
        Bs = torch.randn((sb, cfg.N), device=dev).to(io_t)
        os_ = torch.empty_like(xs)
        for _ in range(5):
            K.ssm_step(xs, ds_, d0["A"], Bs, Bs, d0["D_skip"], xs, hs, out=os_, stream=stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for _ in range(50):
            K.ssm_step(xs, ds_, d0["A"], Bs, Bs, d0["D_skip"], xs, hs, out=os_, stream=stream)
        b.record(stream)
        torch.cuda.synchronize(dev)
        us_call = a.elapsed_time(b) / 50 * 1e3
        # the same 50 steps replayed from a CUDA graph (how a decode loop would issue them): without the host cost
        # of one Python call per launch
        cs = torch.cuda.Stream(dev)
        cs.wait_stream(stream)
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=cs):
            for _ in range(50):
                K.ssm_step(xs, ds_, d0["A"], Bs, Bs, d0["D_skip"], xs, hs, out=os_, stream=cs)
        graph.replay()
        torch.cuda.synchronize(dev)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        graph.replay()
        b.record()
        torch.cuda.synchronize(dev)
        us = a.elapsed_time(b) / 50 * 1e3
        step_bytes = 2 * hs.numel() * 4 + cfg.D * cfg.N * 4 + 4 * xs.numel() * xs.element_size()
        line["decode_step"] = {"batch": sb, "D": cfg.D, "N": cfg.N, "us": us, "us_per_python_call": us_call,
                               "algorithmic_bytes": step_bytes,
                               "achieved_gbs": step_bytes / (us * 1e-6) / 1e9,
                               "frac_of_hbm_peak": step_bytes / (us * 1e-6) / 1e9 / peak,
                               "note": "50 steps replayed from a CUDA graph; state (42 MB) stays in L2 between "
                                       "repetitions"}
    except Exception as exc:  # the headline numbers do not depend on this extra
        line["decode_step"] = {"error": str(exc)}
    # forward only, no checkpoint states written (the prefill use of the scan)
    try:
        if args.no_extras:
            raise RuntimeError("skipped (--no-extras)")
        for i in range(3):
            K.ssm_scan_fwd(sets[i % NSETS]["x"], sets[i % NSETS]["delta"], d0["A"], sets[i % NSETS]["B"],
                           sets[i % NSETS]["C"], d0["D_skip"], sets[i % NSETS]["z"], out=out, stream=stream)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for i in range(20):
            s_ = sets[i % NSETS]
            K.ssm_scan_fwd(s_["x"], s_["delta"], s_["A"], s_["B"], s_["C"], s_["D_skip"], s_["z"], out=out, stream=stream)
        b.record(stream)
        torch.cuda.synchronize(dev)
        p_ms = a.elapsed_time(b) / 20
        line["prefill_fwd"] = {"ms": p_ms, "elements_per_s": cfg.elements / (p_ms * 1e-3),
                               "frac_of_hbm_peak": fwd_bytes / (p_ms * 1e-3) / 1e9 / peak,
                               "note": "ssm_scan_fwd without SSM_FLAG_SAVE_STATES"}
    except Exception as exc:
        line["prefill_fwd"] = {"error": str(exc)}
    # the neighbour of the scan on the SSM branch: short causal depthwise convolution + SiLU (HBM-bound streaming kernels)
    try:
        if args.no_extras:
            raise RuntimeError("skipped (--no-extras)")
        cw = torch.randn((cfg.D, 4), device=dev) * 0.5
        cb = torch.randn((cfg.D,), device=dev) * 0.1
        cy = torch.empty_like(d0["x"])
        cg = {"dx": grads["dx"], "dw": torch.empty_like(cw), "dbias": torch.empty_like(cb)}

        def time_calls(fn, n=30):
            for i in range(5):
                fn(i)
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record(stream)
            for i in range(n):
                fn(i)
            b.record(stream)
            torch.cuda.synchronize(dev)
            return a.elapsed_time(b) / n * 1e3

        f_us = time_calls(lambda i: K.ssm_conv1d_fwd(sets[i % NSETS]["x"], cw, cb, out=cy, stream=stream))
        b_us = time_calls(lambda i: K.ssm_conv1d_bwd(sets[i % NSETS]["x"], cw, cb, sets[i % NSETS]["dout"], outputs=cg,
                                                     stream=stream))
        esz = 2 if cfg.io == "bf16" else 4
        fb, bb = 2 * esz * cfg.elements, 3 * esz * cfg.elements
        line["conv1d"] = {"width": 4, "fwd_us": f_us, "bwd_us": b_us, "fwd_algorithmic_bytes": fb,
                          "bwd_algorithmic_bytes": bb, "fwd_gbs": fb / (f_us * 1e-6) / 1e9,
                          "bwd_gbs": bb / (b_us * 1e-6) / 1e9, "fwd_frac_of_hbm_peak": fb / (f_us * 1e-6) / 1e9 / peak,
                          "bwd_frac_of_hbm_peak": bb / (b_us * 1e-6) / 1e9 / peak,
                          "note": "ssm_conv1d_fwd / ssm_conv1d_bwd (incl. its reduction kernel) on the workload's x and "
                                  "dout, input sets rotated; includes the host cost of one Python call per launch"}
    except Exception as exc:  # the headline numbers do not depend on this extra
        line["conv1d"] = {"error": str(exc)}
    if e2e is not None:
        line["e2e"] = e2e
    if not args.no_extras:
        line["general_A"] = time_shape(K, torch, dev, stream, cfg, peak, general_A=True)
        line["variants"] = {}
        for name, kw in (("zoh", dict(zoh=True)), ("static_bc", dict(static_bc=True)),
                         ("complex_state", dict(complex_state=True))):
            try:
                line["variants"][name] = time_shape(K, torch, dev, stream, cfg, peak, reps=5, **kw)
            except Exception as exc:
                line["variants"][name] = {"error": str(exc)}
        # other state sizes at the same (batch, L, D): N = 8 (bf16: the 16-state kernels on a widened problem) and
        # N = 64 at a quarter of the batch (generic kernels)
        for name, small in (("state_8", cfg.scaled(N=8)), ("state_64_batch_1", cfg.scaled(N=64, batch=1))):
            try:
                line["variants"][name] = time_shape(K, torch, dev, stream, small, peak, reps=5)
            except Exception as exc:
                line["variants"][name] = {"error": str(exc)}
        line["configs"] = {}
        for ci in (1, 2, 4):
            if ci == cfg.cfg_id:
                continue
            try:
                line["configs"][str(ci)] = time_shape(K, torch, dev, stream, synth.CONFIGS[ci], peak)
            except Exception as exc:
                line["configs"][str(ci)] = {"error": str(exc)}
    if not args.no_cpu_baseline and world >= 1:
        line["cpu_baseline"] = cpu_baseline(cfg, host)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


_T0 = time.perf_counter()


def main():
    args = parse_args()
    from paper_2312_00752_b200 import synth
    cfg = synth.CONFIGS[args.config]
    if args.L or args.D:
        cfg = cfg.scaled(L=args.L or cfg.L, D=args.D or cfg.D, name=cfg.name + " (resized)")
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_ours(args, cfg)


if __name__ == "__main__":
    main()
