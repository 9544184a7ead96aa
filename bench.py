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
import json
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
        "tc_phi_forward_k": (Fn * phi1, d * e + Fn * dp * 4, "tensor"),
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
NCU_TRAFFIC_PER_TOKEN_HEAD = {
    "tc_phi_forward_k": 313.5, "tc_state_build": 333.0, "tc_phiq_readout": 477.8, "tc_bwd_query": 305.7, "tc_bwd_key": 594.1,
    "tc_phi_backward_q": 498.8, "tc_phi_backward_k": 619.3,
}


class ClockSampler:
    def __init__(self, index: int):
        self.f = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
        q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
        try:
            self.p = subprocess.Popen(["nvidia-smi", "-i", str(index), f"--query-gpu={q}", "--format=csv,noheader,nounits", "-lms", "20"],
                                      stdout=self.f, stderr=subprocess.DEVNULL)
        except OSError:
            self.p = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": []}
        if self.p is None:
            return out
        self.p.terminate()
        try:
            self.p.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.p.kill()
        self.f.flush()
        self.f.seek(0)
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.f.read().splitlines():
            parts = [x.strip() for x in line.split(",")]
            if len(parts) < 8:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for nm, val in zip(names, parts[4:8]):
                if val.lower().startswith("active"):
                    reasons.add(nm)
        self.f.close()
        os.unlink(self.f.name)
        if sm:
            busy = sorted(sm)[len(sm) // 2:]          # the upper half are the samples under load
            out["sm_mhz"] = float(np.median(busy))
            out["sm_max_mhz"] = float(max(mx))
            out["samples"] = len(sm)
        out["reasons"] = sorted(reasons)
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


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="train_bf16", choices=sorted(synth.CONFIGS))
    ap.add_argument("--B", type=int, default=0, help="override the workload's batch size (profiling on a smaller case)")
    ap.add_argument("--H", type=int, default=0, help="override the workload's head count")
    ap.add_argument("--N", type=int, default=0, help="override the workload's token count")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 0)
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
    tdt = torch.bfloat16 if shape.dtype == "bf16" else torch.float32

    # ---- synthetic inputs (seeded per rank), resident in HBM -----------------------------------------------------
    g = torch.Generator(device=dev)
    g.manual_seed(multi.rank_seed(1000, rank))
    dims = (shape.B, shape.H, shape.N, shape.d)

    def draw():
        return torch.randn(dims, generator=g, device=dev, dtype=torch.float32)

    Q, K, V = draw(), draw(), draw()
    if shape.scale == "inv_sqrt_d":
        s = 1.0 / np.sqrt(shape.d)
        Q, K, V = Q * s, K * s, V * s
    else:
        Q = Q / Q.pow(2).mean(-1, keepdim=True).sqrt()
        K = K / K.pow(2).mean(-1, keepdim=True).sqrt()
    Q, K, V = Q.to(tdt), K.to(tdt), V.to(tdt)
    dO = draw().to(tdt) if shape.backward else None
    pq, pk = synth.make_phi_weights(shape.d, shape.d_phi, shape.F, shape.dtype)
    to_dev = lambda a: torch.from_numpy(a).to(tdt).to(dev)
    pq_d = tuple(to_dev(a) for a in pq)
    pk_d = [tuple(to_dev(a) for a in w) for w in pk]

    op = binding.Hla(shape.B, shape.H, shape.N, shape.d, dtype=shape.dtype, phi="mlp", F=shape.F, d_phi=shape.d_phi, eps=1e-6, device=dev)
    op.set_phi(pq_d, pk_d)
    O = torch.empty_like(V)
    dQ, dK, dV = (torch.empty_like(V) for _ in range(3)) if shape.backward else (None, None, None)
    launches = [0]

    def step():
        binding.hla_forward(op.ctx, Q, K, V, O, op.workspace)
        n = op.launches()
        if shape.backward:
            binding.hla_backward(op.ctx, Q, K, V, O, dO, dQ, dK, dV, op.workspace)
            n += op.launches()
        launches[0] = n

    def barrier():
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 1)):
        step()
    torch.cuda.synchronize()
    if op.device_status() != binding.HLA_OK:
        raise SystemExit("device-side wait timed out during warm-up")

    # ---- timed region: K steps, CUDA events on the launching stream, per-kernel events inside the library -------
    binding.hla_timing_enable(op.ctx, True)
    step()
    torch.cuda.synchronize()
    binding.hla_timing_collect(op.ctx)          # discard: creates the event pool outside the timed region
    sampler = ClockSampler(local)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    e0.record()
    for i in range(args.steps):
        binding.hla_timing_enable(op.ctx, i % 4 == 0)      # per-kernel events on every fourth step: each record stalls the stream ~3 us
        step()
    e1.record()
    barrier()
    ms_total = e0.elapsed_time(e1)
    kt = binding.hla_timing_collect(op.ctx)
    binding.hla_timing_enable(op.ctx, False)
    # The timed region can be shorter than one nvidia-smi sample: keep the same steps running (untimed) until the
    # sampler has had about a second under the same load, then stop it.
    t_tail = time.perf_counter()
    while time.perf_counter() - t_tail < 1.0:
        step()
        torch.cuda.synchronize()
    clocks = sampler.stop()
    clocks["note"] = "sampled over the timed steps and an untimed 1 s tail of the same steps"
    ms_step = multi.max_over_ranks(ms_total, dist, dev) / args.steps
    fl_step, by_step = work_model(shape)
    value = multi.whole_job_rate(fl_step, world, ms_step) / 1e12

    # ---- end to end through the C ABI from pinned host buffers -----------------------------------------------------
    e2e = None
    if not args.no_e2e:
        ins = [Q, K, V] + ([dO] if shape.backward else [])
        outs = [O] + ([dQ, dK, dV] if shape.backward else [])
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

    if rank != 0:
        if dist is not None:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel ------------------------------------------------------------------------------
    peaks = measured_peaks()
    models = kernel_models(shape)
    timed_steps = len(range(0, args.steps, 4))
    per_kernel = {k: {"ms_per_launch": v[0] / v[1], "launches_per_step": v[1] / timed_steps, "share": v[0] / max(sum(x[0] for x in kt.values()), 1e-9)}
                  for k, v in kt.items()}
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
    t_roof = max(by_step / (peaks["hbm"] * 1e9), fl_step / (peaks["tensor"] * 1e12))

    cpu = None
    if not args.no_cpu_baseline and world == 1:
        nh = min(8, shape.B * shape.H)
        dt, fl = oracle_sample(shape, heads=nh)
        cpu = {"value": fl / dt / 1e12, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
               "sample": f"{nh} of {shape.B * shape.H} heads of {shape.name} (N={shape.N}, d={shape.d}), fp64 factored form, {dt:.1f} s"}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": shape.dtype,
            "data": "synthetic",
            "config": {"workload": shape.name, "B": shape.B, "H": shape.H, "N": shape.N, "d": shape.d, "F": shape.F, "d_phi": shape.d_phi,
                       "phi": "mlp", "pass": "fwd+bwd" if shape.backward else "fwd", "parallelism": f"replicas x{world}",
                       "l2": "inputs larger than L2 (each tensor %.0f MB)" % (Q.numel() * Q.element_size() / 1e6)},
            "tokens_per_s": multi.whole_job_rate(shape.B * shape.N, world, ms_step),
            "step_roofline": {"t_roof_ms": t_roof * 1e3, "frac": t_roof * 1e3 / ms_step, "flops": fl_step, "bytes": by_step,
                              "peaks": peaks},
            "roofline": roof, "kernels": per_kernel, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches[0] * args.steps,
            "clocks": clocks}
    print(json.dumps(line), flush=True)
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
