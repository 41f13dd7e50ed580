#!/usr/bin/env python
"""Benchmark of the Representation Shift hot path: a pruned ViT forward pass.

A step is one pass of the whole path (every block: LN, QKV, fused attention,
projection + residual, LN, MLP, residual + shift score, per-sample top-k,
compaction) over one synthetic batch.  One process per GPU; ranks run
independent batches (samples are independent: no exchange step), so N GPUs is
weak scaling and `value` is the sum over ranks.

    python bench.py --gpus 1 --steps 20 --warmup 5
    python bench.py --gpus 4 ...             # starts 4 ranks itself when not launched by torchrun
    python bench.py --impl reference ...     # the fp64 CPU oracle on the host cores

The headline workload is the largest configuration (video ViT-L/14, 4097 tokens); the same JSON
line carries a `workloads` object with the other bf16 configurations.
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

def oracle_sample_plan(wl, target_gflop: float = 400.0):
    """Bounded sample of a workload for the CPU oracle: one block at every distinct token count of
    the schedule, each weighted by the number of blocks that run at that count (a block's cost
    depends on its token count only), on B_s whole samples, B_s chosen so that one pass is about
    `target_gflop` of fp64 work."""
    counts = {}
    for n, r in zip(wl.tokens_per_block(), wl.drops):
        counts.setdefault(n, [0, r])[0] += 1
    per_sample = sum(24.0 * n * wl.D * wl.D + 4.0 * n * n * wl.D for n in counts)
    B_s = int(max(1, min(wl.B, round(target_gflop * 1e9 / per_sample))))
    return B_s, [(n, mult, r) for n, (mult, r) in counts.items()]


class OracleSample:
    """Inputs of the bounded oracle sample; step() runs it once and returns the seconds a whole
    forward of B_s samples takes by that measurement (block time at each count x its multiplicity)."""

    def __init__(self, wl, target_gflop: float = 400.0):
        from paper_2508_00367_b200 import synth
        self.wl = wl
        self.B_s, self.plan = oracle_sample_plan(wl, target_gflop)
        w = synth.make_block_weights(wl.D, wl.D_mlp, wl.dtype, seed=0)
        self.w = {k: v.double().numpy() for k, v in w.items()}
        self.x = {}
        for n, _, _ in self.plan:
            frames = wl.frames if wl.frames and (n - 1) % wl.frames == 0 else 0
            self.x[n] = synth.make_tokens(self.B_s, n, wl.D, wl.dtype, frames, wl.rho, wl.has_cls, seed=n).double().numpy()

    def step(self) -> float:
        from oracle import rs_oracle as orc
        total = 0.0
        for n, mult, r in self.plan:
            t0 = time.perf_counter()
            orc.block_fwd(self.x[n], self.w, self.wl.H, r)
            total += mult * (time.perf_counter() - t0)
        return total

    def describe(self) -> str:
        wl = self.wl
        return (f"{self.B_s} of {wl.B} samples of {wl.name}; one fp64 block (LN, QKV, softmax attention, projection, "
                f"MLP, shift score, top-k, gather) timed at each of the {len(self.plan)} token counts of the schedule, "
                f"each weighted by the number of blocks at that count ({wl.L} blocks in all)")


def time_oracle(wl, steps: int, warmup: int, target_gflop: float = 400.0):
    from oracle import rs_oracle as orc
    smp = OracleSample(wl, target_gflop)
    for _ in range(warmup):
        smp.step()
    t0 = time.perf_counter()
    dt = sum(smp.step() for _ in range(max(steps, 1))) / max(steps, 1)
    wall = (time.perf_counter() - t0) / max(steps, 1)
    return dict(value=smp.B_s / dt, unit=UNIT, cores=orc.num_threads(), kind="oracle", sample=smp.describe(),
                s_per_forward=dt, s_per_step=wall, B_sample=smp.B_s)


def run_reference(args, wl):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    # one sample per step, about a quarter of the default sample: K + W steps end within a few minutes
    res = time_oracle(wl, args.steps, args.warmup, target_gflop=100.0)
    line = dict(metric=METRIC, value=res["value"], unit=UNIT, impl="reference", n_gpus=args.gpus,
                steps=args.steps, warmup=args.warmup, ms_per_step=res["s_per_step"] * 1e3,
                higher_is_better=True, scaling="weak", vs_baseline=None, dtype="f64", data="synthetic",
                config=workload_config(wl, res["B_sample"]),
                cpu_baseline=dict(value=res["value"], unit=UNIT, cores=res["cores"], kind="oracle",
                                  sample=res["sample"]),
                e2e=dict(value=res["value"], unit=UNIT, h2d_bytes_per_step=0, d2h_bytes_per_step=0),
                ms_per_forward=res["s_per_forward"] * 1e3,
                value_from="B_sample / ms_per_forward; ms_per_step is the wall time of one step, which runs each "
                           "distinct token count once (ms_per_forward counts it as often as the schedule has it)")
    print(json.dumps(line))
    return 0


def workload_config(wl, B):
    return dict(workload=wl.name, B_per_gpu=B, N=wl.N, D=wl.D, heads=wl.H, D_mlp=wl.D_mlp, blocks=wl.L,
                drops=list(wl.drops), final_tokens=wl.final_tokens(), storage=wl.dtype,
                l2="4 rotating input batches + per-block weights (working set > 126 MB L2), no flush")


def load_traffic(workload: str, kernel_class: str):
    """DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of a kernel class at a
    workload, from the table of ncu captures under profiles/ (a row is removed there when its kernel
    changes); None when there is no row."""
    path = os.path.join(ROOT, "profiles", "dram_traffic.txt")
    if not os.path.exists(path):
        return None
    for ln in open(path):
        f = ln.split()
        if len(f) >= 3 and not ln.startswith("#") and f[0] == workload and f[1] == kernel_class:
            return float(f[2])
    return None


def pick_bf16_peak(peaks, timed_region_ms: float, clocks):
    """Burst figure when the timed region is short (under a second) or no power cap was seen while it
    ran; the sustained figure for a long region under the cap."""
    capped = bool(clocks) and "sw_power_cap" in (clocks.get("reasons") or [])
    if timed_region_ms < 1000.0 or not capped:
        return peaks["bf16_tflops"], f"{peaks['source']} bf16 burst"
    return peaks["bf16_tflops_sustained"], f"{peaks['source']} bf16 sustained (timed region over 1 s under the power cap)"


def isolated_parts(ctx, wl, peaks, dev):
    """Standalone entry points timed alone (CUDA events around a batch of calls): attention at the
    workload's first-block shape, and the HBM-bound score and select+compact calls on a batch
    scaled up until the working set is several times the L2."""
    import torch

    def bench(fn, iters):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(iters):
            fn()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / iters * 1e-3

    if wl.dtype != "bf16":
        return None
    out = {}
    H, N, D = wl.H, wl.N, wl.D
    qkv = [torch.randn(wl.B, N, 3, H, 64, device=dev).to(torch.bfloat16) for _ in range(3)]
    o = torch.empty(wl.B, N, D, dtype=torch.bfloat16, device=dev)
    cnt = [0]

    def attn():
        cnt[0] += 1
        t = qkv[cnt[0] % 3]
        ctx.attn_fwd(t[:, :, 0], t[:, :, 1], t[:, :, 2], out=o)
    sec = bench(attn, 20)
    fl = 4.0 * wl.B * N * N * D
    out["attn_first_block"] = dict(B=wl.B, N=N, H=H, us=sec * 1e6, tflops=fl / sec / 1e12,
                                   frac_of_bf16_peak=fl / sec / 1e12 / peaks["bf16_tflops"],
                                   note="includes host launch cost when the kernel is shorter than ~25 us")
    del qkv
    Bs = max(wl.B, int(600e6 // (2 * N * D * 2)) + 1)        # two inputs of >= 600 MB together
    a = [torch.randn(Bs, N, D, device=dev).to(torch.bfloat16) for _ in range(2)]
    b = [torch.randn(Bs, N, D, device=dev).to(torch.bfloat16) for _ in range(2)]
    s = torch.empty(Bs, N, dtype=torch.float32, device=dev)

    def score():
        cnt[0] += 1
        ctx.shift_score(a[cnt[0] % 2], b[cnt[0] % 2], out=s)
    sec = bench(score, 10)
    byt = 2 * Bs * N * D * 2 + 4 * Bs * N
    out["score"] = dict(B=Bs, N=N, D=D, mbytes=byt / 1e6, us=sec * 1e6, gbs=byt / sec / 1e9,
                        frac_of_hbm_peak=byt / sec / 1e9 / peaks["hbm_gbs"])
    r = max(1, wl.drops[0] if wl.drops[0] > 0 else max(wl.drops))
    K = N - r
    xo = torch.empty(Bs, K, D, dtype=torch.bfloat16, device=dev)
    ki = torch.empty(Bs, K, dtype=torch.int32, device=dev)

    def compact():
        cnt[0] += 1
        ctx.topk_compact(s, a[cnt[0] % 2], r, True, x_out=xo, keep_idx=ki)
    sec = bench(compact, 10)
    byt = 4 * Bs * N + 4 * Bs * K + 2 * Bs * K * D * 2
    out["select_compact"] = dict(B=Bs, N=N, D=D, r=r, mbytes=byt / 1e6, us=sec * 1e6, gbs=byt / sec / 1e9,
                                 frac_of_hbm_peak=byt / sec / 1e9 / peaks["hbm_gbs"])
    del a, b, xo
    # line-wise pruning of a feature map (Sec. 4, CNN): the first-stage output of a ResNet-50 on 224 x 224
    # images, 56 x 56 positions of 256 channels, 8 rows and 8 columns removed; batch scaled past the L2
    Hh, Ww, Dc, dr, dc = 56, 56, 256, 8, 8
    Bl = int(600e6 // (Hh * Ww * Dc * 2)) + 1
    fm = [torch.randn(Bl, Hh, Ww, Dc, device=dev).to(torch.bfloat16) for _ in range(2)]
    ls = torch.rand(Bl, Hh, Ww, device=dev)
    lo = torch.empty(Bl, Hh - dr, Ww - dc, Dc, dtype=torch.bfloat16, device=dev)
    lr = torch.empty(Bl, Hh - dr, dtype=torch.int32, device=dev)
    lc = torch.empty(Bl, Ww - dc, dtype=torch.int32, device=dev)

    def linewise():
        cnt[0] += 1
        ctx.linewise_compact(ls, fm[cnt[0] % 2], dr, dc, x_out=lo, keep_rows=lr, keep_cols=lc)
    sec = bench(linewise, 10)
    byt = 4 * Bl * Hh * Ww + 2 * Bl * (Hh - dr) * (Ww - dc) * Dc * 2
    out["linewise_compact"] = dict(B=Bl, H=Hh, W=Ww, D=Dc, drop_rows=dr, drop_cols=dc, mbytes=byt / 1e6, us=sec * 1e6,
                                   gbs=byt / sec / 1e9, frac_of_hbm_peak=byt / sec / 1e9 / peaks["hbm_gbs"])
    return out


# ------------------------------------------------------------------ GPU arm

NBUF = 4      # rotating input batches


def measure_workload(ctx, wl, args, dev, rank, world, headline: bool, sampler=None):
    """Times one workload on this rank.  Always: the resident step (graph replay unless --no-graph)
    and the per-kernel-class device time of an eager pass.  For the headline also the end-to-end
    step from pinned host memory."""
    import torch
    import torch.distributed as dist
    import paper_2508_00367_b200 as rs
    from paper_2508_00367_b200 import synth

    tdt = torch.bfloat16 if wl.dtype == "bf16" else torch.float32
    x0, blocks = synth.make_workload(wl, seed=0)
    # only the final tokens are materialised; LN1 of the blocks that follow a non-pruning block is applied inside
    # their QKV product (rs_prepare_ln1_fold) unless --no-ln-fold
    model = rs.PrunedViT(ctx, blocks, wl.H, list(wl.drops), tdt, tap_blocks=[], fold_ln1=not args.no_ln_fold)
    del blocks
    gen = torch.Generator().manual_seed(100 + rank)
    host_x = [x0.to(tdt).pin_memory()] + [
        synth.make_tokens(wl.B, wl.N, wl.D, wl.dtype, wl.frames, wl.rho, wl.has_cls, gen=gen).to(tdt).pin_memory()
        for _ in range(NBUF - 1)]
    dev_x = [h.to(dev) for h in host_x]
    host_out = torch.empty((wl.B, wl.final_tokens(), wl.D), dtype=tdt).pin_memory()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps, tail=None):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for i in range(steps):
            fn(i)
        if tail is not None:
            tail()                        # whatever the steps left running on other streams ends inside the region
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

    warm = max(args.warmup, 3)
    for i in range(max(warm, NBUF)):      # every input buffer's graph exists before the timed region
        step_resident(i)
    ctx.async_status()

    if sampler is not None:
        sampler.start()
    n0 = ctx.launch_count()
    ms = timed(step_resident, args.steps)
    launches = ctx.launch_count() - n0
    if use_graph:      # replays do not pass through the library's counter: kernels per captured forward x steps
        launches = model.launches_per_forward(wl.B, wl.N, wl.D) * args.steps
    clocks = sampler.stop() if sampler is not None else None
    res = dict(ms=ms, launches=int(launches), clocks=clocks)

    if headline:
        # End to end: host buffers in, host buffer out, through the same public call.  The upload of
        # a step's input and the download of the previous step's result run on a copy stream while
        # a forward computes (two device input buffers; the result leaves through two device staging
        # buffers, because the model's own output buffer is overwritten by the next forward).
        dxs = [torch.empty_like(dev_x[0]) for _ in range(2)]
        copy_stream = torch.cuda.Stream(device=dev)          # uploads
        down_stream = torch.cuda.Stream(device=dev)          # downloads (a stream of their own: they wait for a forward)
        ev_in = [torch.cuda.Event() for _ in range(2)]      # upload into dxs[k] finished
        ev_free = [torch.cuda.Event() for _ in range(2)]    # forward reading dxs[k] finished
        stage = [torch.empty_like(host_out, device=dev) for _ in range(2)]
        ev_out = [torch.cuda.Event() for _ in range(2)]     # result copied into stage[k]
        ev_down = [torch.cuda.Event() for _ in range(2)]    # stage[k] read out to the host

        def step_e2e(i):
            k = i % 2
            main = torch.cuda.current_stream(dev)
            with torch.cuda.stream(copy_stream):
                copy_stream.wait_event(ev_free[k])
                dxs[k].copy_(host_x[i % NBUF], non_blocking=True)
                ev_in[k].record(copy_stream)
            main.wait_event(ev_in[k])
            outs = model.forward(dxs[k], graph=use_graph)
            ev_free[k].record(main)
            main.wait_event(ev_down[k])
            stage[k].copy_(outs[-1]["x_out"], non_blocking=True)
            ev_out[k].record(main)
            with torch.cuda.stream(down_stream):
                down_stream.wait_event(ev_out[k])
                host_out.copy_(stage[k], non_blocking=True)
                ev_down[k].record(down_stream)

        for k in range(2):
            ev_free[k].record(torch.cuda.current_stream(dev))
            ev_down[k].record(torch.cuda.current_stream(dev))
        for i in range(4):
            step_e2e(i)
        res["ms_e2e"] = timed(step_e2e, args.steps, tail=lambda: torch.cuda.current_stream(dev).wait_stream(down_stream))
        res["h2d"] = host_x[0].numel() * host_x[0].element_size()
        res["d2h"] = host_out.numel() * host_out.element_size()

    # Per-kernel-class device time: a separate eager pass in which the library brackets every
    # launch with CUDA events on the launch stream.  The events cost a few microseconds per launch
    # (and keep a kernel's set-up from overlapping its predecessor), so the plain eager step is
    # timed too and the difference, spread evenly over the launches, is reported beside the raw sums.
    tsteps = min(args.steps, 5)
    ms_eager = timed(lambda i: model.forward(dev_x[i % NBUF]), tsteps)
    ctx.timing_enable(True)
    for i in range(tsteps):
        model.forward(dev_x[i % NBUF])
    per = ctx.timing_read()
    ctx.timing_enable(False)
    ctx.async_status()
    n_launch = sum(v["launches"] for v in per.values()) / tsteps
    raw_ms = {k: v["ms"] / tsteps for k, v in per.items()}
    ev_us = max(0.0, (sum(raw_ms.values()) - ms_eager) / max(n_launch, 1.0) * 1e3)
    res.update(ms_eager=ms_eager, raw_ms=raw_ms, ev_us=ev_us,
               cls_launches={k: per[k]["launches"] // tsteps for k in per},
               cls_ms={k: (max(raw_ms[k] - per[k]["launches"] / tsteps * ev_us * 1e-3, 1e-9) if per[k]["launches"] else 0.0)
                       for k in per},
               tensor_cores=bool(ctx.uses_tensor_cores(tdt)), use_graph=use_graph)
    del model, dev_x, host_x
    torch.cuda.empty_cache()
    return res


def class_report(wl, m, peak_tf):
    """Throughput of the two tensor-core kernel classes of a measured workload: algorithmic FLOP of
    the pruned schedule / event-timed class time, raw and with the event overhead taken off."""
    Ns = wl.tokens_per_block()
    out = {}
    for cls, fl in (("gemm", gemm_flops(wl.B, Ns, wl.D, wl.D_mlp)), ("attn", attn_flops(wl.B, Ns, wl.D))):
        raw, cor = m["raw_ms"][cls], m["cls_ms"][cls]
        out[cls] = dict(gflop_per_step=fl / 1e9, launches_per_step=m["cls_launches"][cls], ms_per_step=raw,
                        tflops=fl / (raw * 1e-3) / 1e12, frac=fl / (raw * 1e-3) / 1e12 / peak_tf,
                        ms_per_step_overhead_corrected=cor, tflops_overhead_corrected=fl / (cor * 1e-3) / 1e12,
                        frac_overhead_corrected=fl / (cor * 1e-3) / 1e12 / peak_tf)
    return out


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

    m = measure_workload(ctx, wl, args, dev, rank, world, True, ClockSampler(local) if rank == 0 else None)
    others = {}
    if world == 1 and not args.no_other_workloads:
        for name, w2 in synth.WORKLOADS.items():
            if w2.dtype == "bf16" and name != wl.name:
                others[name] = (w2, measure_workload(ctx, w2, args, dev, rank, world, False))

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return 0

    peaks = load_peaks()
    Ns = wl.tokens_per_block()
    gf = gemm_flops(wl.B, Ns, wl.D, wl.D_mlp)
    af = attn_flops(wl.B, Ns, wl.D)
    ms, clocks = m["ms"], m["clocks"]
    peak_tf, peak_src = pick_bf16_peak(peaks, ms * args.steps, clocks)
    cr = class_report(wl, m, peak_tf)
    dom = "gemm" if m["raw_ms"]["gemm"] >= m["raw_ms"]["attn"] else "attn"
    kname = {"gemm": "gemm_tc_kernel (QKV, proj, FC1, FC2; every launch of a step)",
             "attn": "attn_tc_kernel (every launch of a step)"}[dom]
    d = cr[dom]
    roofline = dict(bound="tensor", kernel=kname, achieved=d["tflops"], peak=peak_tf, unit="TFLOP/s", frac=d["frac"],
                    peak_source=peak_src, traffic=load_traffic(wl.name, dom), tensor_cores=m["tensor_cores"],
                    launches_per_step=d["launches_per_step"], ms_per_step=d["ms_per_step"],
                    gflop_per_step=d["gflop_per_step"],
                    achieved_overhead_corrected=d["tflops_overhead_corrected"],
                    frac_overhead_corrected=d["frac_overhead_corrected"],
                    event_overhead_us_per_launch=m["ev_us"], eager_ms_per_step=m["ms_eager"],
                    frac_of_nominal_2250=d["tflops"] / 2250.0,
                    timing="per-launch CUDA events on the launch stream in an eager pass; achieved = gflop_per_step / "
                           "ms_per_step (the events' own cost included); *_overhead_corrected takes (sum of event-timed "
                           "launches - plain eager step) / launches off every launch")
    sz = 2 if wl.dtype == "bf16" else 4
    gather_bytes = sum(2 * wl.B * (n - r) * wl.D * sz for n, r in zip(Ns, wl.drops) if r > 0)
    # pruning blocks before the last write no dense copy of their kept tokens (read in place by the next block)
    # (with the LayerNorm fold the kept rows are copied, un-normalised, instead of their LN1 being written: the same bytes)
    dense_copy_bytes_removed = (sum(wl.B * (n - r) * wl.D * sz for n, r in list(zip(Ns, wl.drops))[:-1] if r > 0)
                                if args.no_ln_fold or wl.dtype != "bf16" else 0)
    cls_ms = m["cls_ms"]
    other_cls = "attn" if dom == "gemm" else "gemm"
    parts = {
        other_cls: cr[other_cls],
        "attn_target_0p60_met": bool(cr["attn"]["frac"] >= 0.60),
        "attn_kernels": "attn_tc_kernel (two query tiles per CTA) or attn_tc3_kernel (three, 64-key tiles), "
                        "whichever the library's cost model expects to be faster for the block's B, N and H",
        "attn_kernel_by_tokens": {str(n): rs.attn_kernel_choice(torch.cuda.get_device_properties(dev).multi_processor_count,
                                                                 wl.B, wl.H, n) for n in sorted(set(Ns), reverse=True)},
        "gather": dict(ms_per_step=m["raw_ms"]["gather"], ms_per_step_overhead_corrected=cls_ms["gather"],
                       gbs=(gather_bytes / (m["raw_ms"]["gather"] * 1e-3) / 1e9 if m["raw_ms"]["gather"] else 0.0),
                       dense_copy_bytes_not_written_per_step=dense_copy_bytes_removed,
                       note=("selection, index lists and LN1 of the next block in one kernel for N <= 4608; the dense "
                             "[B, K, D] copy is written for the last block only") if args.no_ln_fold else
                            ("selection, index lists, the kept rows and their sums (LN1 of the next block is applied "
                             "inside its QKV product)")),
        "select": dict(ms_per_step=m["raw_ms"]["select"]),
        "layernorm": dict(ms_per_step=m["raw_ms"]["layernorm"]),
        "note": "in-situ, event-timed; activations between kernels sit in the 126 MB L2 "
                "(L2-assisted GB/s); the shift score rides in the FC2 epilogue (no kernel of its own)",
        "isolated": isolated_parts(ctx, wl, peaks, dev) if not args.no_isolated else None,
    }

    workloads = {}
    for name, (w2, m2) in others.items():
        c2 = class_report(w2, m2, peaks["bf16_tflops"])
        N2 = w2.tokens_per_block()
        fl2 = gemm_flops(w2.B, N2, w2.D, w2.D_mlp) + attn_flops(w2.B, N2, w2.D)
        workloads[name] = dict(B=w2.B, N=w2.N, blocks=w2.L, final_tokens=w2.final_tokens(), ms_per_step=m2["ms"],
                               samples_per_s=w2.B / (m2["ms"] * 1e-3), model_tflops=fl2 / (m2["ms"] * 1e-3) / 1e12,
                               gpu_launches_per_step=m2["launches"] // args.steps, gemm=c2["gemm"], attn=c2["attn"],
                               other_ms_per_step={k: m2["raw_ms"][k] for k in ("layernorm", "select", "gather")},
                               peak="bf16 burst (every timed region here is under a second)")

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        r = time_oracle(wl, 1, 0)
        cpu = dict(value=r["value"], unit=UNIT, cores=r["cores"], kind="oracle", sample=r["sample"])

    value = aggregate_throughput(wl.B, ms, world)
    line = dict(metric=METRIC, value=value, unit=UNIT, n_gpus=world, steps=args.steps, warmup=max(args.warmup, 3),
                ms_per_step=ms, higher_is_better=True, scaling="weak", vs_baseline=None,
                dtype=("bf16" if wl.dtype == "bf16" else "f32"), data="synthetic",
                config=dict(workload_config(wl, wl.B), launch=("CUDA graph replay, one graph per input buffer" if m["use_graph"] else "host launches")), clocks=clocks,
                e2e=dict(value=aggregate_throughput(wl.B, m["ms_e2e"], world), unit=UNIT,
                         h2d_bytes_per_step=m["h2d"], d2h_bytes_per_step=m["d2h"], ms_per_step=m["ms_e2e"]),
                gpu_launches=int(m["launches"]), roofline=roofline, kernels=parts, cpu_baseline=cpu,
                model_tflops=(gf + af) / (ms * 1e-3) / 1e12, workloads=workloads)
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()
    return 0


# ------------------------------------------------------------------ launch

def spawn_ranks(n: int, cmd, port: int = 0, extra_env=None, timeout=None):
    """Start `cmd` n times as ranks 0..n-1 of one job on this node (RANK, LOCAL_RANK, WORLD_SIZE,
    MASTER_ADDR = 127.0.0.1, MASTER_PORT in the environment) and wait for all of them.  Returns the
    list of return codes; rank 0 inherits stdout, so its one JSON line is the job's."""
    import socket
    if not port:
        with socket.socket() as sk:
            sk.bind(("127.0.0.1", 0))
            port = sk.getsockname()[1]
    env = dict(os.environ, WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    env.update(extra_env or {})
    procs = [subprocess.Popen(list(cmd), env=dict(env, RANK=str(r), LOCAL_RANK=str(r)),
                              stdout=(None if r == 0 else subprocess.DEVNULL)) for r in range(n)]
    rcs = []
    for p in procs:
        try:
            rcs.append(p.wait(timeout=timeout))
        except subprocess.TimeoutExpired:
            p.kill()
            rcs.append(-9)
    return rcs


def main(argv=None):
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="video_vit_l14")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the `workloads` object (the other bf16 configurations)")
    ap.add_argument("--no-isolated", action="store_true", help="skip the stand-alone attention / score / compaction timings")
    ap.add_argument("--no-ln-fold", action="store_true", help="keep LN1 a kernel of its own in every block")
    ap.add_argument("--no-graph", action="store_true", help="launch every kernel from the host instead of replaying a CUDA graph")
    args = ap.parse_args(argv)
    from paper_2508_00367_b200 import synth
    wl = synth.WORKLOADS[args.workload]
    world_env = os.environ.get("WORLD_SIZE")
    if args.gpus > 1 and world_env is None:
        # not under torchrun: start the ranks here (one process per GPU, independent batches)
        rcs = spawn_ranks(args.gpus, [sys.executable, os.path.abspath(__file__)] + list(sys.argv[1:] if argv is None else argv))
        return max(abs(rc) for rc in rcs)
    if world_env is not None and int(world_env) != args.gpus:
        print(f"bench.py: --gpus {args.gpus} but WORLD_SIZE={world_env}", file=sys.stderr)
        return 2
    if args.impl == "reference":
        return run_reference(args, wl)
    return run_gpu(args, wl)


if __name__ == "__main__":
    sys.exit(main())
