"""CPU-only checks of the host side: the shared library loads and exports every
symbol the header declares, the package's schedule tables reproduce the counts
the paper's printed GFLOPs imply, and batch sharding across ranks (the only
multi-GPU mode: independent samples, no exchange step) is a partition."""
import ctypes
import os
import re
import subprocess
import sys

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    import glob
    names = set()
    for h in glob.glob(os.path.join(ROOT, "include", "*.h")):
        names |= set(re.findall(r"RS_API[^;(]*?\b(rs_[a-z_0-9]+)\s*\(", open(h).read()))
    return sorted(names)


def test_library_builds_and_exports_every_declared_symbol():
    from paper_2508_00367_b200 import build, binding
    lib_path = build.build()
    lib = ctypes.CDLL(lib_path)
    names = _declared()
    assert len(names) >= 11
    for n in names:
        assert hasattr(lib, n), n
    for n in binding.EXPORTS:
        assert n in names


def test_workspace_query_needs_no_gpu():
    from paper_2508_00367_b200 import binding
    lib = binding.load_library()
    d = binding.BlockDesc(1, 1, 64, 197, 768, 12, 3072, 16, 1, 0.0, 0.0, 0, 0)
    n = lib.rs_block_workspace_bytes(ctypes.byref(d))
    T = 64 * 197
    assert n >= T * 768 * 2 * (1 + 3 + 1) + T * 3072 * 2     # u, qkv, o, h at least
    bad = binding.BlockDesc(7, 1, 64, 197, 768, 12, 3072, 16, 1, 0.0, 0.0, 0, 0)
    assert lib.rs_block_workspace_bytes(ctypes.byref(bad)) == 0


def test_vit_workspace_query_needs_no_gpu():
    from paper_2508_00367_b200 import binding
    lib = binding.load_library()
    d = binding.VitDesc(1, 64, 197, 768, 12, 3072, 3, 1, 0.0, 0.0, 0, 0)
    drops = (ctypes.c_int * 3)(16, 0, 16)
    n = lib.rs_vit_workspace_bytes(ctypes.byref(d), drops)
    blk = lib.rs_block_workspace_bytes(ctypes.byref(binding.BlockDesc(1, 1, 64, 197, 768, 12, 3072, 16, 1, 0.0, 0.0, 0, 0)))
    assert n >= blk + 2 * 64 * 197 * 768 * 2          # largest block scratch + two token buffers
    bad = (ctypes.c_int * 3)(16, 0, 181)               # the last block would drop all of its 181 tokens
    assert lib.rs_vit_workspace_bytes(ctypes.byref(d), bad) == 0


def test_workload_schedules():
    from paper_2508_00367_b200 import synth
    w = synth.WORKLOADS
    assert w["vit_s_block"].tokens_per_block() == [197] and w["vit_s_block"].final_tokens() == 181
    assert w["vit_b16"].tokens_per_block() == [197 - 16 * i for i in range(12)] and w["vit_b16"].final_tokens() == 5
    assert w["vit_l16_384"].tokens_per_block()[-1] == 117 and w["vit_l16_384"].final_tokens() == 97
    t = w["video_vit_b16"].tokens_per_block()
    assert (t[0], t[3], t[6], t[9], w["video_vit_b16"].final_tokens()) == (1569, 1099, 770, 539, 539)
    t = w["video_vit_l14"].tokens_per_block()
    assert (t[0], t[4], t[8], t[12], t[16], t[23]) == (4097, 3073, 2305, 1729, 1297, 1297)


def test_video_tokens_are_ar1():
    from paper_2508_00367_b200 import synth
    x = synth.make_tokens(4, 1 + 8 * 196, 64, "f32", frames=8, rho=0.9, seed=3)
    fr = x[:, 1:].reshape(4, 8, 196, 64)
    assert abs(fr.std().item() - 1.0) < 0.02
    a, b = fr[:, :-1].flatten(), fr[:, 1:].flatten()
    rho = torch.corrcoef(torch.stack([a, b]))[0, 1].item()
    assert abs(rho - 0.9) < 0.01
    # bf16 storage: values are exactly representable
    xb = synth.make_tokens(1, 197, 64, "bf16", seed=3)
    assert torch.equal(xb, xb.to(torch.bfloat16).float())


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    from paper_2508_00367_b200 import binding
    monkeypatch.setattr(binding, "_lib", None)
    monkeypatch.setattr(binding, "LIB_PATH", str(tmp_path / "nope.so"))
    with pytest.raises(RuntimeError):
        binding.load_library()


_WORKER = r"""
import os, sys, torch, torch.distributed as dist
sys.path.insert(0, sys.argv[1])
import bench
dist.init_process_group("gloo", rank=int(os.environ["RANK"]), world_size=int(os.environ["WORLD_SIZE"]))
rank, world = dist.get_rank(), dist.get_world_size()
lo, hi = bench.shard_range(64, rank, world)
mine = torch.zeros(64); mine[lo:hi] = 1
dist.all_reduce(mine)
assert torch.equal(mine, torch.ones(64)), mine          # every sample owned exactly once
t = torch.tensor([10.0 + rank]); dist.all_reduce(t, op=dist.ReduceOp.MAX)
assert t.item() == 10.0 + world - 1                      # max-over-ranks timing reduction
val = bench.aggregate_throughput(hi - lo, t.item(), world)
print("OK", rank, lo, hi, val)
dist.destroy_process_group()
"""


def test_batch_sharding_two_ranks_gloo(tmp_path):
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29581", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, str(script), ROOT], env=dict(env, RANK=str(r)),
                              stdout=subprocess.PIPE, stderr=subprocess.STDOUT, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120)[0] for p in procs]
    for p, o in zip(procs, outs):
        assert p.returncode == 0, o
        assert "OK" in o


def test_bench_spawns_its_own_ranks(tmp_path):
    """`bench.py --gpus N` outside torchrun starts N ranks itself: spawn_ranks gives every child its
    rank and one rendezvous; here two CPU ranks meet over gloo and shard a batch."""
    sys.path.insert(0, ROOT)
    import bench
    script = tmp_path / "worker.py"
    script.write_text(_WORKER)
    marks = tmp_path / "ranks"
    marks.mkdir()
    wrapper = tmp_path / "wrap.py"
    wrapper.write_text("import os, sys, runpy\n"
                       f"open(os.path.join({str(marks)!r}, os.environ['RANK'] + '_' + os.environ['LOCAL_RANK'] + '_' + os.environ['WORLD_SIZE']), 'w').close()\n"
                       f"sys.argv = [{str(script)!r}, {ROOT!r}]\n"
                       f"runpy.run_path({str(script)!r}, run_name='__main__')\n")
    rcs = bench.spawn_ranks(2, [sys.executable, str(wrapper)], timeout=120)
    assert rcs == [0, 0]
    assert sorted(os.listdir(marks)) == ["0_0_2", "1_1_2"]
    # a WORLD_SIZE that contradicts --gpus is an error, not a silent one-rank run
    env = dict(os.environ, WORLD_SIZE="2", RANK="0", LOCAL_RANK="0")
    p = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "4", "--impl", "reference"],
                       env=env, capture_output=True, text=True, timeout=120)
    assert p.returncode == 2 and "WORLD_SIZE" in p.stderr


def test_per_device_once_guard(tmp_path):
    """Kernel attributes are per device: the guard that sets them runs the set-up once for every
    device, again after a failure, and never caches an out-of-range device index."""
    src = tmp_path / "once.cpp"
    src.write_text(r"""
#include "rs_once.h"
#include <thread>
#include <vector>
#include <cstdio>
int main() {
    rs::PerDeviceOnce once;
    int calls[3] = {0, 0, 0};
    for (int rep = 0; rep < 3; ++rep)
        for (int dev = 0; dev < 2; ++dev)
            if (once.run(dev, [&] { ++calls[dev]; return 0; }) != 0) return 1;
    if (calls[0] != 1 || calls[1] != 1) return 2;                 // once per device, not once per process
    if (!once.done(0) || !once.done(1) || once.done(2)) return 3;
    int fails = 0;
    if (once.run(2, [&] { ++fails; return 7; }) != 7) return 4;   // a failed set-up is reported ...
    if (once.done(2)) return 5;
    if (once.run(2, [&] { ++calls[2]; return 0; }) != 0 || calls[2] != 1 || !once.done(2)) return 6;   // ... and retried
    int n = 0;
    once.run(-1, [&] { ++n; return 0; });
    once.run(1000, [&] { ++n; return 0; });
    once.run(1000, [&] { ++n; return 0; });
    if (n != 3) return 7;                                          // never cached outside the table
    rs::PerDeviceOnce shared;
    int hits = 0;
    std::vector<std::thread> th;
    for (int t = 0; t < 8; ++t) th.emplace_back([&] { for (int i = 0; i < 1000; ++i) shared.run(5, [&] { ++hits; return 0; }); });
    for (auto& t : th) t.join();
    if (hits != 1) return 8;
    std::puts("ok");
    return 0;
}
""")
    exe = tmp_path / "once"
    csrc = os.path.join(ROOT, "paper_2508_00367_b200", "csrc")
    subprocess.check_call(["g++", "-std=c++17", "-O1", "-pthread", "-I", csrc, "-o", str(exe), str(src)])
    p = subprocess.run([str(exe)], capture_output=True, text=True)
    assert p.returncode == 0 and p.stdout.strip() == "ok", (p.returncode, p.stdout)


def test_static_status_before_any_static_call_needs_no_gpu_work():
    """Header contract: arguments are validated on the host; a null descriptor is refused."""
    from paper_2508_00367_b200 import binding
    lib = binding.load_library()
    err = ctypes.create_string_buffer(128)
    st = lib.rs_block_fwd_static(None, None, None, None, None, None, None, None, err, 128)
    assert st == 1 and b"null" in err.value


def test_gelu_polynomial_matches_exact_erf_gelu():
    """The FC1 epilogue's GELU constants come from csrc/fit_gelu.py: refit and check the bound
    the kernel's comment states (fp32 Horner evaluation against the erf definition)."""
    import importlib.util
    import re
    here = os.path.dirname(os.path.abspath(__file__))
    csrc = os.path.join(os.path.dirname(here), "paper_2508_00367_b200", "csrc")
    spec = importlib.util.spec_from_file_location("fit_gelu", os.path.join(csrc, "fit_gelu.py"))
    fg = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(fg)
    import numpy as np
    coef = fg.fit()
    assert fg.max_error_fp32(coef) < 1e-6
    assert coef[-1] > 0                       # 2^-q -> 0 for large |v|
    # the constants compiled into the kernel are these coefficients
    src = open(os.path.join(csrc, "rs_gemm_tc.cu")).read()
    body = src[src.index("float gelu_erf(float v)"):]
    body = body[:body.index("return v *")]
    consts = [float(m) for m in re.findall(r"(-?\d+\.\d+(?:e-?\d+)?)f", body)]
    in_kernel = np.array(consts[:6][::-1], dtype=np.float64)     # Horner order is highest degree first
    assert fg.max_error_fp32(in_kernel) < 1e-6


def test_attention_kernel_choice_follows_the_measured_winners():
    """The cost model that picks between the two attention kernels (two or three query tiles per thread
    block) against the kernel that was the faster one when both were timed on a B200 of 148 SMs (CUDA
    events over graph replays; the one shape the model gets wrong, B=4 H=16 N=2305, lost 3 %)."""
    import paper_2508_00367_b200 as rs
    measured = {  # (B, H, N): faster kernel
        (4, 16, 4097): 3, (4, 16, 3073): 3, (4, 16, 1729): 2, (4, 16, 1297): 3, (16, 12, 1569): 3, (16, 12, 1099): 3,
        (16, 12, 770): 3, (16, 12, 539): 2, (32, 16, 577): 3, (32, 16, 337): 3, (64, 12, 197): 2, (1, 16, 4097): 2,
    }
    for (B, H, N), want in measured.items():
        assert rs.attn_kernel_choice(148, B, H, N) == want, (B, H, N)
    assert rs.attn_kernel_choice(148, 4, 16, 2305) == 2          # measured 151.5 against 147.1 us: the known miss
    for N in (1, 64, 128):
        assert rs.attn_kernel_choice(148, 64, 12, N) == 2        # one query tile per head: two heads per item
    assert rs.attn_kernel_choice(0, 1, 1, 1) == 0

