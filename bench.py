#!/usr/bin/env python
"""Benchmark of the Representation Shift hot path: a pruned ViT forward pass.

A step is one pass of the whole path (every block: LN, QKV, fused attention,
projection + residual, LN, MLP, residual + shift score, per-sample top-k,
compaction) over one synthetic batch.  One process per GPU; ranks run
independent batches (samples are independent: no exchange step), so N GPUs is
weak scaling and `value` is the sum over ranks.

    python bench.py --gpus 1 --steps 20 --warmup 5
    python bench.py --impl reference ...     # the fp64 CPU oracle on the host cores
"""
from __future__ import annotations

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

METRIC = "pruned_vit_forward_throughput"
UNIT = "samples/s"


# ------------------------------------------------------------------ host helpers (CPU-tested)

def shard_range(total: int, rank: int, world: int):
    """Contiguous slice of `total` samples owned by `rank` (sizes differ by at most 1)."""
    base, rem = divmod(total, world)
    lo = rank * base + min(rank, rem)
    return lo, lo + base + (1 if rank < rem else 0)


def aggregate_throughput(samples_per_rank_per_step: int, ms_per_step_max: float, world: int) -> float:
    """Whole-job samples/s: every rank did `samples_per_rank_per_step` per step; time = max over ranks."""
    return world * samples_per_rank_per_step / (ms_per_step_max * 1e-3)


def gemm_flops(B, Ns, D, Dm):
    return sum(2 * B * n * (3 * D * D + D * D + 2 * D * Dm) for n in Ns)


def attn_flops(B, Ns, D):
    return sum(4 * B * n * n * D for n in Ns)


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        d = json.load(open(p))
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons with nvidia-smi while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.rows, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append(line.strip())

    def stop(self):
        if not self.proc:
            return dict(sm_mhz=None, sm_max_mhz=None, reasons=["nvidia-smi unavailable"])
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in self.rows:
            f = [t.strip() for t in r.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        sm.sort()
        return dict(sm_mhz=(sm[len(sm) // 2] if sm else None), sm_max_mhz=(max(mx) if mx else None),
                    power_w_max=(max(power) if power else None), samples=len(sm), reasons=sorted(reasons))


# ------------------------------------------------------------------ reference arm: the CPU oracle

def time_oracle(wl, B_sample: int, steps: int, warmup: int):
    import numpy as np
    from oracle import rs_oracle as orc
    from paper_2508_00367_b200 import synth
    x, blocks = synth.make_workload(wl, seed=0, B=B_sample)
    xn = x.double().numpy()
    wn = [{k: v.double().numpy() for k, v in w.items()} for w in blocks]
    io = "bf16" if wl.dtype == "bf16" else "f32"
    for _ in range(warmup):
        orc.model_fwd(xn, wn, wl.H, list(wl.drops), io_dtype=io)
    t0 = time.perf_counter()
    for _ in range(steps):
        orc.model_fwd(xn, wn, wl.H, list(wl.drops), io_dtype=io)
    dt = (time.perf_counter() - t0) / max(steps, 1)
    return dict(value=B_sample / dt, unit=UNIT, cores=orc.num_threads(), kind="oracle",
                sample=f"{B_sample} of {wl.B} samples of {wl.name}, whole {wl.L}-block pruned forward, fp64",
                s_per_step=dt)


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    res = time_oracle(wl, 1, args.steps, args.warmup)
    line = dict(metric=METRIC, value=res["value"], unit=UNIT, impl="reference", n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=res["s_per_step"] * 1e3,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=workload_config(wl, 1),
                cpu_baseline=dict(value=res["value"], unit=UNIT, cores=res["cores"], kind="oracle",
                                  sample=res["sample"]),
                e2e=dict(value=res["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0))
    print(json.dumps(line))
    return 0


def workload_config(wl, B):
    return dict(workload=wl.name, B_per_gpu=B, N=wl.N, D=wl.D, heads=wl.H, D_mlp=wl.D_mlp, blocks=wl.L,
                drops=list(wl.drops), final_tokens=wl.final_tokens(), storage=wl.dtype,
                l2="4 rotating input batches + per-block weights (working set > 126 MB L2), no flush")


# ------------------------------------------------------------------ GPU arm

def run_gpu(args, wl):
    import torch
    import torch.distributed as dist
    import paper_2508_00367_b200 as rs
    from paper_2508_00367_b200 import synth

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32

    ctx = rs.Context(local)
    x0, blocks = synth.make_workload(wl, seed=0)
    model = rs.PrunedViT(ctx, blocks, wl.H, list(wl.drops), tdt)
    NBUF = 4
    gen = torch.Generator().manual_seed(100 + rank)
    host_x = [x0.to(tdt).pin_memory()] + [
        synth.make_tokens(wl.B, wl.N, wl.D, wl.dtype, wl.frames, wl.rho, wl.has_cls, gen=gen).to(tdt).pin_memory()
        for _ in range(NBUF - 1)]
    dev_x = [h.to(dev) for h in host_x]
    final_shape = (wl.B, wl.final_tokens(), wl.D)
    host_out = torch.empty(final_shape, dtype=tdt).pin_memory()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            fn(i)
        e1.record()
        torch.cuda.synchronize()
        ms = e0.elapsed_time(e1) / steps
        if world > 1:
            t = torch.tensor([ms], device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            ms = float(t.item())
        barrier()
        return ms

    use_graph = not args.no_graph

    def step_resident(i):
        model.forward(dev_x[i % NBUF], graph=use_graph)

    dx = torch.empty_like(dev_x[0])

    def step_e2e(i):
        dx.copy_(host_x[i % NBUF], non_blocking=True)
        outs = model.forward(dx, graph=use_graph)
        host_out.copy_(outs[-1]["x_out"], non_blocking=True)

    for i in range(max(args.warmup, 3)):
        step_resident(i)
    ctx.async_status()

    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
    n0 = ctx.launch_count()
    ms = timed(step_resident, args.steps)
    launches = ctx.launch_count() - n0
    if use_graph:      # replays do not pass through the library's counter: kernels per captured forward x steps
        launches = model.launches_per_forward(wl.B, wl.N, wl.D) * args.steps
    clocks = sampler.stop() if rank == 0 else None

    for i in range(3):
        step_e2e(i)
    ms_e2e = timed(step_e2e, args.steps)

    # per-kernel-class device time, separate pass so the events do not sit in the headline timing
    ctx.timing_enable(True)
    tsteps = min(args.steps, 5)
    for i in range(tsteps):
        model.forward(dev_x[i % NBUF])        # eager: the per-launch events are recorded by the library
    per = ctx.timing_read()
    ctx.timing_enable(False)
    ctx.async_status()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peaks = load_peaks()
    Ns = wl.tokens_per_block()
    gf = gemm_flops(wl.B, Ns, wl.D, wl.D_mlp)
    af = attn_flops(wl.B, Ns, wl.D)
    gemm_ms = per["gemm"]["ms"] / tsteps
    attn_ms = per["attn"]["ms"] / tsteps
    tc = ctx.uses_tensor_cores(tdt)
    peak_tf = peaks["bf16_tflops_sustained"]
    achieved = gf / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    roofline = dict(bound="tensor", kernel="gemm (QKV, proj, FC1, FC2; all launches of a step)",
                    achieved=achieved, peak=peak_tf, unit="TFLOP/s", frac=achieved / peak_tf,
                    peak_source=f"{peaks['source']} bf16 sustained", traffic=None,
                    tensor_cores=bool(tc), launches_per_step=per["gemm"]["launches"] // tsteps,
                    ms_per_step=gemm_ms)
    sz = 2 if wl.dtype == "bf16" else 4
    score_bytes = sum(wl.B * n * (wl.D * 4 * 2 + wl.D * sz + 4) for n in Ns)
    gather_bytes = sum(2 * wl.B * (n - r) * wl.D * sz for n, r in zip(Ns, wl.drops) if r > 0)
    parts = {
        "attn": dict(ms_per_step=attn_ms, tflops=(af / (attn_ms * 1e-3) / 1e12 if attn_ms > 0 else 0.0),
                     frac_of_bf16_peak=(af / (attn_ms * 1e-3) / 1e12 / peaks["bf16_tflops"] if attn_ms > 0 else 0.0)),
        "score": dict(ms_per_step=per["score"]["ms"] / tsteps,
                      gbs=score_bytes / (per["score"]["ms"] / tsteps * 1e-3) / 1e9 if per["score"]["ms"] > 0 else 0.0),
        "gather": dict(ms_per_step=per["gather"]["ms"] / tsteps,
                       gbs=gather_bytes / (per["gather"]["ms"] / tsteps * 1e-3) / 1e9 if per["gather"]["ms"] > 0 else 0.0),
        "select": dict(ms_per_step=per["select"]["ms"] / tsteps),
        "layernorm": dict(ms_per_step=per["layernorm"]["ms"] / tsteps),
        "note": "in-situ event timing; score/gather working sets fit the 126 MB L2 (L2-assisted GB/s)",
    }

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        Bs = {"vit_s_block": 2, "vit_b16": 4, "vit_l16_384": 1, "video_vit_b16": 1, "video_vit_l14": 1}[wl.name]
        r = time_oracle(wl, Bs, 1, 0)
        cpu = dict(value=r["value"], unit=UNIT, cores=r["cores"], kind="oracle", sample=r["sample"])

    value = aggregate_throughput(wl.B, ms, world)
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype=("bf16" if wl.dtype == "bf16" else "f32"), data="synthetic",
                config=dict(workload_config(wl, wl.B), launch=("CUDA graph replay, one graph per input buffer" if use_graph else "host launches")), clocks=clocks,
                e2e=dict(value=aggregate_throughput(wl.B, ms_e2e, world), unit=UNIT,
                         h2d_bytes_per_step=host_x[0].numel() * host_x[0].element_size(),
                         d2h_bytes_per_step=host_out.numel() * host_out.element_size(), ms_per_step=ms_e2e),
                gpu_launches=int(launches), roofline=roofline, kernels=parts, cpu_baseline=cpu,
                model_tflops=(gf + af) / (ms * 1e-3) / 1e12)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="vit_b16")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying a CUDA graph")
    args = ap.parse_args()
    from paper_2508_00367_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    if args.impl == "reference":
        return run_reference(args, wl)
    return run_gpu(args, wl)


if __name__ == "__main__":
    sys.exit(main())
