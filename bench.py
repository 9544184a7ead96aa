#!/usr/bin/env python
"""Benchmark of the HLA operator (forward + backward) on synthetic video-DiT-shaped inputs.

    python bench.py --gpus N --steps K --warmup W [--impl reference] [--workload NAME]

One "step" is one pass of the whole hot path over one batch: hla_forward followed by
hla_backward (forward only for the workloads that have no backward).  Rank 0 prints ONE
JSON line.  With N > 1 (launched by torch.distributed.run) every rank runs the same
per-GPU workload on its own seeded inputs - batches are independent, so there is no
collective on the data path (weak scaling) - and `value` aggregates all ranks over the
slowest rank's device time.
"""
from __future__ import annotations

import argparse
import datetime
import json
import math
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_12128_b200 import flops as F_, multi, synth  # noqa: E402

METRIC = "hla_fwd_bwd_tflops"
UNIT = "TFLOP/s"
FP32_ALU_TFLOPS = 148 * 128 * 2 * 1.965e9 / 1e12     # 148 SMs x 128 FMA lanes x 2 flop x max SM clock


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        p = json.load(open(path))
        return {"hbm": p["hbm_gbs"], "tensor": p["bf16_tflops_sustained"], "src": "measured"}
    return {"hbm": 6650.0, "tensor": 1400.0, "src": "fallback"}


def work_model(shape):
    """Algorithmic FLOPs and HBM bytes of one step, whole job on one GPU."""
    th = shape.B * shape.H * shape.N
    fl = F_.fwd_flops_per_token(shape.d, shape.F, shape.d_phi)
    by = F_.fwd_bytes_per_token(shape.d, shape.F, shape.d_phi)
    if shape.backward:
        fl += F_.bwd_flops_per_token(shape.d, shape.F, shape.d_phi)
        by += F_.bwd_bytes_per_token(shape.d, shape.F, shape.d_phi)
    return th * fl, th * by


def kernel_models(shape):
    """Per launch: (algorithmic flops, algorithmic HBM bytes, compute unit) of each kernel; the per-token-head
    figures are FLOPs = 2 x multiply-adds of the paper's factored scheme and the tensors each kernel must stream once.
    Tiny kernels (reductions) are left out."""
    d, P, dp, Fn = shape.d, shape.d_phi ** shape.F, shape.d_phi, shape.F
    th = shape.B * shape.H * shape.N
    e = 2
    contr = 2 * P * (d + 1)
    phi1 = 2 * d * (d + dp)
    m = {
        "tc_state_build": (contr, d * e + Fn * dp * 4, "tensor"),
        "tc_readout": (contr, d * e + dp * 4 + 4, "tensor"),
        "tc_phiq_readout": (phi1 + contr, 2 * d * e + dp * 4 + 4, "tensor"),      # phi_q + readout + normaliser in one kernel
        "tc_phik_state": (Fn * phi1 + contr, 2 * d * e + Fn * dp * 4, "tensor"),       # phi_k1..F + state build in one kernel
        "tc_bwd_query": (2 * contr, 2 * d * e + 3 * dp * 4, "tensor"),
        "tc_bwd_key": (2 * contr, 2 * d * e + 2 * Fn * dp * 4, "tensor"),
        "tc_phi_backward_q": (4 * d * d + 2 * d * dp, 2 * d * e + 2 * dp * 4, "tensor"),
        "tc_phi_backward_k": (Fn * (4 * d * d + 2 * d * dp), 2 * d * e + 2 * Fn * dp * 4, "tensor"),
        "simt_phi_forward": ((1 + Fn) * phi1 / 2, d * e + (1 + Fn) * dp * 2, "alu"),          # two launches: Q side, K side
        "simt_state_build": (contr, 2 * d * e + Fn * dp * 4, "alu"),
        "simt_readout": (contr, d * e + Fn * dp * 4, "alu"),
        "simt_feature_grad": (contr, 2 * d * e + 2 * Fn * dp * 4, "alu"),
        "simt_phi_backward": ((1 + Fn) * (4 * d * d + 2 * d * dp) / 2, 2 * d * e + (1 + Fn) * dp * 2, "alu"),
    }
    return {k: (v[0] * th, v[1] * th, v[2]) for k, v in m.items()}


# DRAM traffic per token-head of a launch (dram__bytes_read.sum + dram__bytes_write.sum of one ncu capture,
# scaled by token-heads; see profiles/).  None = not captured yet.
NCU_TRAFFIC_PER_TOKEN_HEAD = {"tc_phik_state": 586.7, "tc_state_build": 333.0, "tc_phiq_readout": 476.9, "tc_bwd_query": 304.3, "tc_bwd_key": 594.3,
                              "tc_phi_backward_q": 499.6, "tc_phi_backward_k": 616.1}


class ClockSampler:
    """nvidia-smi polled in the background.  Every sample carries its own time stamp, so the samples that fall inside a
    window of the run (sustained warm-up + timed region) can be picked afterwards; of those, the ones with a GPU
    utilisation above 50 % are the samples under load."""
    FIELDS = ("timestamp,clocks.sm,clocks.max.sm,power.draw,utilization.gpu,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    REASONS = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "20"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None
        self.rows = None

    def stop(self):
        if self.rows is not None:
            return
        self.rows = []
        if self.p is None:
            return
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 9:
                continue
            try:
                t = datetime.datetime.strptime(parts[0], "%Y/%m/%d %H:%M:%S.%f").timestamp()
                self.rows.append((t, float(parts[1]), float(parts[2]), float(parts[3]), float(parts[4]),
                                  [nm for nm, val in zip(self.REASONS, parts[5:9]) if val.lower().startswith("active")]))
            except ValueError:
                continue
        self.f.close()
        os.unlink(self.f.name)

    def window(self, t0: float, t1: float) -> dict:
        """Summary of the samples stamped in [t0, t1] (host clock, seconds)."""
        self.stop()
        rows = [r for r in self.rows if t0 <= r[0] <= t1]
        busy = [r for r in rows if r[4] > 50.0]
        out = {"sm_mhz": None, "sm_min_mhz": None, "sm_max_mhz": None, "power_w": None, "reasons": [], "samples": len(rows),
               "samples_under_load": len(busy), "note": "samples stamped inside the sustained warm-up and the timed region; under load = utilisation > 50 %"}
        use = busy or rows
        if use:
            out["sm_mhz"] = float(np.median([r[1] for r in use]))
            out["sm_min_mhz"] = float(min(r[1] for r in use))
            out["sm_max_mhz"] = float(max(r[2] for r in use))
            out["power_w"] = float(np.median([r[3] for r in use]))
            out["reasons"] = sorted({nm for r in use for nm in r[5]})
        return out


def oracle_sample(shape, heads=1, seed=0):
    """The fp64 oracle (factored form, as it stands) on `heads` heads of the workload; returns (seconds, flops)."""
    from oracle import hla_oracle as orc
    sub = synth.HlaShape("sample", 1, heads, shape.N, shape.d, shape.dtype, shape.scale, shape.backward, shape.F, shape.d_phi)
    Q, K, V = (a.astype(np.float64) for a in synth.make_qkv(sub, seed))
    pq, pk = synth.make_phi_weights(shape.d, shape.d_phi, shape.F, shape.dtype)
    dO = synth.make_dO(sub).astype(np.float64)
    t0 = time.perf_counter()
    orc.hla_forward(Q, K, V, pq, pk, 1e-6, "factored")
    if shape.backward:
        orc.hla_backward(Q, K, V, dO, pq, pk, 1e-6, "factored")
    dt = time.perf_counter() - t0
    fl, _ = work_model(sub)
    return dt, fl


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [i.get("num_threads", 1) for i in threadpool_info() if i.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return len(os.sched_getaffinity(0))


def run_reference(args, shape, rank, world):
    """The reference arm: the CPU oracle on the GPU machine's host cores, each step a one-head sample of the workload."""
    if rank != 0:
        return
    times = []
    fl = 0
    for i in range(args.warmup + args.steps):
        dt, fl = oracle_sample(shape, heads=1, seed=i)
        if i >= args.warmup:
            times.append(dt)
    ms = 1e3 * float(np.mean(times))
    val = fl / (ms * 1e-3) / 1e12
    cores = blas_threads()
    sample = f"1 head of {shape.name} (B=1,H=1,N={shape.N},d={shape.d}) per step, fp64, factored form"
    line = {"impl": "reference", "metric": METRIC, "value": val, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": shape.name, "B": shape.B, "H": shape.H, "N": shape.N, "d": shape.d, "F": shape.F,
                                            "d_phi": shape.d_phi, "sample": sample},
            "cpu_baseline": {"value": val, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": val, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "tokens_per_s": shape.N / (ms * 1e-3), "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def roofline_of(shape, ms_step, world, peaks):
    """Step roofline.  `frac` uses the work the hardware has to do: the larger of the algorithmic HBM bytes at the copy
    bandwidth and the FLOPs of the symmetry-folded scheme (what the kernels execute) at the tensor peak.
    `frac_algorithmic` is the same with the paper's unfolded FLOP count (P = d_phi^F features per contraction), which
    the kernels never issue; it is kept as a labelled second figure."""
    fl_alg, by = work_model(shape)
    th = shape.B * shape.H * shape.N
    fl_exec = th * F_.folded_flops_per_token(shape.d, shape.F, shape.d_phi, shape.backward)
    t_mem = by / (peaks["hbm"] * 1e9)
    t_exec = fl_exec / (peaks["tensor"] * 1e12)
    t_alg = fl_alg / (peaks["tensor"] * 1e12)
    t_roof = max(t_mem, t_exec)
    return {"t_roof_ms": t_roof * 1e3, "frac": t_roof * 1e3 / ms_step, "bound": "hbm" if t_mem >= t_exec else "tensor",
            "t_hbm_ms": t_mem * 1e3, "t_tensor_executed_ms": t_exec * 1e3, "t_tensor_algorithmic_ms": t_alg * 1e3,
            "frac_algorithmic": max(t_mem, t_alg) * 1e3 / ms_step, "flops_algorithmic": fl_alg, "flops_executed": fl_exec, "bytes": by,
            "peaks": peaks}


class Workload:
    """One configuration resident in HBM: synthetic inputs (seeded per rank), the operator context and its outputs."""

    def __init__(self, shape, rank, dev):
        import torch
        from paper_2602_12128_b200 import binding
        self.torch, self.binding, self.shape, self.dev = torch, binding, shape, dev
        tdt = torch.bfloat16 if shape.dtype == "bf16" else torch.float32
        g = torch.Generator(device=dev)
        g.manual_seed(multi.rank_seed(1000, rank))
        dims = (shape.B, shape.H, shape.N, shape.d)

        def draw():
            return torch.randn(dims, generator=g, device=dev, dtype=torch.float32)

        Q, K, V = draw(), draw(), draw()
        if shape.scale == "inv_sqrt_d":
            sc = 1.0 / np.sqrt(shape.d)
            Q, K, V = Q * sc, K * sc, V * sc
        else:
            Q = Q / Q.pow(2).mean(-1, keepdim=True).sqrt()
            K = K / K.pow(2).mean(-1, keepdim=True).sqrt()
        self.Q, self.K, self.V = Q.to(tdt), K.to(tdt), V.to(tdt)
        self.dO = draw().to(tdt) if shape.backward else None
        del Q, K, V
        pq, pk = synth.make_phi_weights(shape.d, shape.d_phi, shape.F, shape.dtype)
        to_dev = lambda a: torch.from_numpy(a).to(tdt).to(dev)
        self.op = binding.Hla(shape.B, shape.H, shape.N, shape.d, dtype=shape.dtype, phi="mlp", F=shape.F, d_phi=shape.d_phi, eps=1e-6, device=dev,
                              causal=shape.causal)
        self.op.set_phi(tuple(to_dev(a) for a in pq), [tuple(to_dev(a) for a in w) for w in pk])
        self.O = torch.empty_like(self.V)
        self.dQ, self.dK, self.dV = (torch.empty_like(self.V) for _ in range(3)) if shape.backward else (None, None, None)
        self.launches = 0

    def step(self):
        b, op = self.binding, self.op
        b.hla_forward(op.ctx, self.Q, self.K, self.V, self.O, op.workspace)
        n = op.launches()
        if self.shape.backward:
            b.hla_backward(op.ctx, self.Q, self.K, self.V, self.O, self.dO, self.dQ, self.dK, self.dV, op.workspace)
            n += op.launches()
        self.launches = n

    def timed(self, nsteps):
        """Device time of `nsteps` steps enqueued back to back (CUDA events on the launching stream), in ms."""
        torch = self.torch
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(nsteps):
            self.step()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    def sustain(self, seconds, ms_estimate):
        """The same steps, untimed and without host synchronisation, for about `seconds` of device time, so that the
        clocks settle under the power cap before anything is timed."""
        n = int(min(max(math.ceil(seconds * 1e3 / max(ms_estimate, 1e-3)), 1), 50000))
        for _ in range(n):
            self.step()
        return n

    def kernel_times(self, nsteps):
        """Per-kernel device time from event records inside the library, on steps of their own (the records stall the
        stream a few microseconds each, so they stay out of every timed region)."""
        b, op = self.binding, self.op
        b.hla_timing_enable(op.ctx, True)
        self.step()
        self.torch.cuda.synchronize()
        b.hla_timing_collect(op.ctx)            # discard: creates the event pool
        for _ in range(nsteps):
            self.step()
        self.torch.cuda.synchronize()
        kt = b.hla_timing_collect(op.ctx)
        b.hla_timing_enable(op.ctx, False)
        return kt


def value_mod_leg(shape, w, dev, short=False):
    """hla_value_mod_forward (+ backward for workloads with a backward) on the workload's O and V, sustained like the rest
    (short: three calls only, for a profiler capture)."""
    import torch
    from paper_2602_12128_b200 import binding
    tdt = torch.bfloat16
    rng = np.random.default_rng(9)
    d = shape.d

    def vmlp():
        r = lambda *s: torch.from_numpy(rng.standard_normal(s).astype(np.float32))
        ws = (1.0 + 0.2 * r(d), 0.1 * r(d), r(d, d) / np.sqrt(d), 0.1 * r(d), r(d, d) / np.sqrt(d), 0.1 * r(d))
        return tuple(x.to(tdt).to(dev) for x in ws)

    op = binding.Hla(shape.B, shape.H, shape.N, d, dtype="bf16", phi="none", eps=1e-6, device=dev, value_mod=True)
    op.set_phi_v(vmlp(), vmlp())
    out = torch.empty_like(w.O)
    dT, dV = (torch.empty_like(w.O), torch.empty_like(w.O)) if shape.backward else (None, None)

    def step():
        binding.hla_value_mod_forward(op.ctx, w.O, w.V, out, op.workspace)
        n = op.launches()
        if shape.backward:
            binding.hla_value_mod_backward(op.ctx, w.O, w.V, w.dO, dT, dV, False, op.workspace)
            n += op.launches()
        return n

    for _ in range(3):
        launches = step()
    torch.cuda.synchronize()
    if op.device_status() != binding.HLA_OK:
        raise SystemExit("device-side wait timed out (value modulation)")
    if short:
        return None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(5):
        step()
    e1.record()
    torch.cuda.synchronize()
    est = e0.elapsed_time(e1) / 5
    n = int(min(max(math.ceil(500.0 / est), 10), 20000))
    for _ in range(n):
        step()
    e0.record()
    for _ in range(n):
        step()
    e1.record()
    torch.cuda.synchronize()
    ms = e0.elapsed_time(e1) / n
    th = shape.B * shape.H * shape.N
    fl = th * F_.value_mod_flops_per_token(d, shape.backward)
    by = th * d * 2 * (3 + (4 if shape.backward else 0))      # T, V in, Out out (+ dOut in, dT, dV out, and T, V again)
    return {"ms_per_step": ms, "steps": n, "tflops": fl / (ms * 1e-3) / 1e12, "gpu_launches_per_step": launches, "flops": fl, "bytes": by,
            "pass": "fwd+bwd" if shape.backward else "fwd",
            "note": "hla_value_mod_forward (+ _backward): FLOPs = the 4 (+ 4) d x d products per token; the backward's recomputed forward is not counted"}


def extra_leg(name, rank, dev, peaks, local):
    """One of the other configurations, timed by the same code: >= 1 s of untimed sustained steps, then >= 0.5 s timed."""
    import torch
    from paper_2602_12128_b200 import binding
    shape = synth.CONFIGS[name]
    w = Workload(shape, rank, dev)
    for _ in range(3):
        w.step()
    torch.cuda.synchronize()
    if w.op.device_status() != binding.HLA_OK:
        raise SystemExit(f"device-side wait timed out ({name})")
    est = w.timed(5) / 5
    sampler = ClockSampler(local)
    t0 = time.time()
    w.sustain(1.0, est)
    n = int(min(max(math.ceil(500.0 / est), 10), 50000))
    ms = w.timed(n) / n
    t1 = time.time()
    clocks = sampler.window(t0, t1)
    fl, _ = work_model(shape)
    roof = roofline_of(shape, ms, 1, peaks)
    roof.pop("peaks")
    out = {"config": {"B": shape.B, "H": shape.H, "N": shape.N, "d": shape.d, "pass": "fwd+bwd" if shape.backward else "fwd", "causal": bool(shape.causal)},
           "ms_per_step": ms, "steps": n, "tflops": fl / (ms * 1e-3) / 1e12, "tokens_per_s": shape.B * shape.N / (ms * 1e-3),
           "gpu_launches_per_step": w.launches, "step_roofline": roof,
           "clocks": {k: clocks[k] for k in ("sm_mhz", "sm_min_mhz", "power_w", "reasons", "samples_under_load")}}
    if clocks["sm_mhz"]:
        out["ms_x_mhz"] = ms * clocks["sm_mhz"]
    del w
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="train_bf16", choices=sorted(synth.CONFIGS))
    ap.add_argument("--B", type=int, default=0, help="override the workload's batch size (profiling on a smaller case)")
    ap.add_argument("--H", type=int, default=0, help="override the workload's head count")
    ap.add_argument("--N", type=int, default=0, help="override the workload's token count")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extra", action="store_true", help="skip the other configurations (the `extra` object of the line)")
    ap.add_argument("--profile", action="store_true", help="only warm-up and the timed steps: no sustained phase, no extra legs (for ncu)")
    ap.add_argument("--also", default="", help="with --profile: comma list of side calls to run three times after the steps "
                    "(weights = hla_backward_weights, vmod = hla_value_mod_forward/backward), so that a capture can name their kernels")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
    if args.profile:
        args.no_e2e = args.no_cpu_baseline = args.no_extra = True
    shape = synth.CONFIGS[args.workload]
    if args.B or args.H or args.N:
        import dataclasses
        shape = dataclasses.replace(shape, name=shape.name + "_resized", B=args.B or shape.B, H=args.H or shape.H, N=args.N or shape.N)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.impl == "reference":
        run_reference(args, shape, rank, world)
        return

    import torch
    from paper_2602_12128_b200 import binding

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (the CUDA library has no CPU fallback)")
    torch.cuda.set_device(local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    dev = torch.device("cuda", local)
    peaks = measured_peaks()

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    w = Workload(shape, rank, dev)
    op = w.op
    for _ in range(max(args.warmup, 1)):
        w.step()
    torch.cuda.synchronize()
    if op.device_status() != binding.HLA_OK:
        raise SystemExit("device-side wait timed out during warm-up")

    # ---- sustained untimed steps (>= 1 s, no host synchronisation), then the timed region: exactly K steps ------------
    est = w.timed(3) / 3
    sampler = ClockSampler(local)
    t_win0 = time.time()
    n_sustain = 0 if args.profile else w.sustain(1.0, est)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for _ in range(args.steps):
        w.step()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    # a longer run of the same steps right behind it: the steady-state figure (>= 0.5 s of device time)
    ms_steady, n_steady = None, 0
    if not args.profile:
        n_steady = int(min(max(math.ceil(500.0 / est), args.steps), 50000))
        ms_steady = w.timed(n_steady) / n_steady
    t_win1 = time.time()
    clocks = sampler.window(t_win0, t_win1)
    n_kt = max(8, n_steady)          # as long as the steady run, so the per-kernel times are taken under the same clocks
    kt = {} if args.profile else w.kernel_times(n_kt)
    ms_step = multi.max_over_ranks(ms_total, dist, dev) / args.steps
    if ms_steady is not None:
        ms_steady = multi.max_over_ranks(ms_steady, dist, dev)
    fl_step, by_step = work_model(shape)
    value = multi.whole_job_rate(fl_step, world, ms_step) / 1e12

    # ---- end to end through the C ABI from pinned host buffers -----------------------------------------------------
    e2e = None
    if not args.no_e2e:
        ins = [w.Q, w.K, w.V] + ([w.dO] if shape.backward else [])
        outs = [w.O] + ([w.dQ, w.dK, w.dV] if shape.backward else [])
        h_in = [torch.empty(x.shape, dtype=x.dtype, pin_memory=True).copy_(x) for x in ins]
        h_out = [torch.empty(x.shape, dtype=x.dtype, pin_memory=True) for x in outs]
        nsteps = max(2, min(args.steps, 6))
        # Every step copies its inputs from pinned host memory and its results back.  The copies of neighbouring steps
        # overlap (PCIe is full duplex): two sets of device buffers, one stream each for copy-in, compute and copy-out.
        sets_in = [ins, [torch.empty_like(x) for x in ins]]
        sets_out = [outs, [torch.empty_like(x) for x in outs]]
        s_in, s_cmp, s_out = (torch.cuda.Stream(device=dev) for _ in range(3))
        ev_in = [torch.cuda.Event() for _ in range(2)]
        ev_cmp = [torch.cuda.Event() for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]

        def e2e_step(i):
            k = i & 1
            bi, bo = sets_in[k], sets_out[k]
            with torch.cuda.stream(s_in):
                s_in.wait_event(ev_cmp[k])                 # the compute that last read this input set has finished
                for d_, h_ in zip(bi, h_in):
                    d_.copy_(h_, non_blocking=True)
                ev_in[k].record(s_in)
            with torch.cuda.stream(s_cmp):
                s_cmp.wait_event(ev_in[k])
                s_cmp.wait_event(ev_out[k])                # the copy-out that last read this output set has finished
                binding.hla_forward(op.ctx, bi[0], bi[1], bi[2], bo[0], op.workspace, s_cmp)
                if shape.backward:
                    binding.hla_backward(op.ctx, bi[0], bi[1], bi[2], bo[0], bi[3], bo[1], bo[2], bo[3], op.workspace, s_cmp)
                ev_cmp[k].record(s_cmp)
            with torch.cuda.stream(s_out):
                s_out.wait_event(ev_cmp[k])
                for d_, h_ in zip(bo, h_out):
                    h_.copy_(d_, non_blocking=True)
                ev_out[k].record(s_out)

        barrier()
        for i in range(2):
            e2e_step(i)
        barrier()
        e0.record(s_in)
        for i in range(nsteps):
            e2e_step(i)
        e1.record(s_out)
        barrier()
        ms_e2e = multi.max_over_ranks(e0.elapsed_time(e1), dist, dev) / nsteps
        e2e = {"value": multi.whole_job_rate(fl_step, world, ms_e2e) / 1e12, "unit": UNIT, "ms_per_step": ms_e2e, "steps": nsteps,
               "h2d_bytes_per_step": int(sum(x.numel() * x.element_size() for x in ins)),
               "d2h_bytes_per_step": int(sum(x.numel() * x.element_size() for x in outs))}
        del h_in, h_out, sets_in, sets_out

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel ------------------------------------------------------------------------------
    models = kernel_models(shape)
    tot_k = max(sum(x[0] for x in kt.values()), 1e-9)
    per_kernel = {k: {"ms_per_launch": v[0] / v[1], "launches_per_step": v[1] / n_kt, "share": v[0] / tot_k} for k, v in kt.items()}
    roof = None
    if kt:
        top = max(kt, key=lambda k: kt[k][0])
        dur = kt[top][0] / kt[top][1] * 1e-3
        if top in models:
            fl, by, unit = models[top]
            comp_peak = peaks["tensor"] if unit == "tensor" else FP32_ALU_TFLOPS
            t_mem, t_comp = by / (peaks["hbm"] * 1e9), fl / (comp_peak * 1e12)
            if t_mem >= t_comp:
                roof = {"bound": "hbm", "achieved": by / dur / 1e9, "peak": peaks["hbm"], "unit": "GB/s"}
            else:
                roof = {"bound": unit, "achieved": fl / dur / 1e12, "peak": comp_peak, "unit": "TFLOP/s"}
            roof["frac"] = roof["achieved"] / roof["peak"]
            tr = NCU_TRAFFIC_PER_TOKEN_HEAD.get(top)
            roof["traffic"] = None if tr is None else tr * shape.B * shape.H * shape.N
            roof["kernel"] = top
            roof["peak_source"] = peaks["src"] if roof["bound"] != "alu" else "derived: 148 SM x 128 lanes x 2 x 1.965 GHz"
            roof["ms_per_launch"] = dur * 1e3
            roof["flops_per_launch"] = fl
            roof["bytes_per_launch"] = by

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        nh = min(8, shape.B * shape.H)
        dt, fl = oracle_sample(shape, heads=nh)
        cpu = {"value": fl / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"{nh} of {shape.B * shape.H} heads of {shape.name} (N={shape.N}, d={shape.d}), numpy fp64 factored form with BLAS threads, {dt:.1f} s"}

    # ---- gradients of the phi weights (a separate call after the backward; not part of `value`) ------------------------
    wgrad = None
    if shape.backward and not args.profile and world == 1:
        gq, gk = op.backward_weights(w.Q, w.K)        # allocates the outputs once
        torch.cuda.synchronize()

        def wstep():
            binding.hla_backward_weights(op.ctx, w.Q, w.K, gq, gk, op.workspace)

        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(5):
            wstep()
        ev1.record()
        torch.cuda.synchronize()
        est_w = ev0.elapsed_time(ev1) / 5
        n_w = int(min(max(math.ceil(500.0 / est_w), 10), 20000))
        for _ in range(n_w):                          # untimed, to settle the clocks
            wstep()
        ev0.record()
        for _ in range(n_w):
            wstep()
        ev1.record()
        torch.cuda.synchronize()
        ms_w = ev0.elapsed_time(ev1) / n_w
        fl_w = shape.B * shape.H * shape.N * (1 + shape.F) * (2 * shape.d * shape.d + 2 * shape.d * shape.d_phi)
        wgrad = {"ms_per_call": ms_w, "calls": n_w, "tflops": fl_w / (ms_w * 1e-3) / 1e12, "gpu_launches_per_call": op.launches(),
                 "flops": fl_w, "note": "hla_backward_weights: dW1, db1, dW2, db2 of phi_q and phi_k1..F; FLOPs = the two weight-gradient "
                 "products per map (the recomputed hidden layer is not counted)"}
        del gq, gk

    if args.profile and world == 1:
        also = [a for a in args.also.split(",") if a]
        if "weights" in also and shape.backward:
            gq, gk = op.backward_weights(w.Q, w.K)
            for _ in range(2):
                binding.hla_backward_weights(op.ctx, w.Q, w.K, gq, gk, op.workspace)
            torch.cuda.synchronize()
        if "vmod" in also:
            value_mod_leg(shape, w, dev, short=True)

    # ---- value modulation of the attention result (Section 4.5; separate calls, not part of `value`) --------------------
    vmod = None
    if not args.profile and world == 1 and shape.dtype == "bf16" and shape.d in (64, 128):
        vmod = value_mod_leg(shape, w, dev)

    tensor_mb = w.Q.numel() * w.Q.element_size() / 1e6
    launches_per_step = w.launches
    # ---- the other configurations, timed by the same code (single-GPU runs only) ----------------------------------------
    extra = None
    if not args.no_extra and world == 1:
        del w, op
        torch.cuda.empty_cache()
        extra = {}
        for name in ("long_bf16", "dit_bf16", "small_bf16", "paper_r1_bf16", "paper_r2_bf16", "train_bf16_2f", "train_bf16_causal"):
            if name != shape.name:
                extra[name] = extra_leg(name, rank, dev, peaks, local)

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "ms_per_step_steady": ms_steady, "steady_steps": n_steady, "sustained_untimed_steps": n_sustain,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": shape.dtype,
            "data": "synthetic",
            "config": {"workload": shape.name, "B": shape.B, "H": shape.H, "N": shape.N, "d": shape.d, "F": shape.F, "d_phi": shape.d_phi,
                       "phi": "mlp", "pass": "fwd+bwd" if shape.backward else "fwd", "parallelism": f"replicas x{world}",
                       "l2": "inputs larger than L2 (each tensor %.0f MB)" % tensor_mb},
            "tokens_per_s": multi.whole_job_rate(shape.B * shape.N, world, ms_step),
            "step_roofline": roofline_of(shape, ms_step, world, peaks),
            "roofline": roof, "kernels": per_kernel, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches_per_step * args.steps,
            "clocks": clocks, "weight_gradients": wgrad, "value_modulation": vmod, "extra": extra}
    if clocks.get("sm_mhz"):
        line["ms_x_mhz"] = ms_step * clocks["sm_mhz"]
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
