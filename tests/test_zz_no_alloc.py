"""rs_block_fwd_static -- the block for callers that cannot allocate device memory
where they call it (inside a serving loop that must not hit cudaMalloc, or a plug-in
that only receives its input and output buffers).  Its scratch is an array built into
the library, shared by all calls on a device.

The test drives the entry point through the C ABI twice in a row, with different
inputs, and requires the same results as rs_block_fwd with a caller workspace (the
kernels are the same, so the comparison is exact); a third call repeats the first
input to show that what earlier calls left in the shared scratch does not matter.
This file sorts last so that a failure here cannot hide any other test."""
import ctypes

import pytest
import torch

from paper_2508_00367_b200 import synth


def test_oversized_block_is_rejected_without_touching_the_gpu():
    from paper_2508_00367_b200 import binding
    lib = binding.load_library()
    assert lib.rs_static_scratch_bytes() == 16 << 20
    d = binding.BlockDesc(1, 1, 64, 197, 768, 12, 3072, 16, 1, 0.0, 0.0, 0, 0)   # needs ~400 MB
    w = binding.BlockWeights()
    err = ctypes.create_string_buffer(256)
    st = lib.rs_block_fwd_static(ctypes.byref(d), ctypes.byref(w), None, None, None, None, None, None, err, 256)
    assert st == 3 and b"built-in array holds" in err.value


@pytest.mark.gpu
@pytest.mark.parametrize("dtype,B,N,D,H,r", [("f32", 2, 197, 384, 6, 16), ("bf16", 2, 197, 768, 12, 16)])
def test_static_scratch_block_matches_workspace_block(dtype, B, N, D, H, r):
    import paper_2508_00367_b200 as rs
    tdt = torch.float32 if dtype == "f32" else torch.bfloat16
    ctx = rs.Context(0)
    w = synth.make_block_weights(D, 4 * D, dtype, seed=21)
    dw = rs.DeviceBlockWeights(w, tdt, ctx.device)
    xs = [synth.make_tokens(B, N, D, dtype, seed=s).to(tdt).cuda() for s in (31, 32)]
    want = [ctx.block_fwd(x, dw, H, r, want_full=True) for x in xs]
    got = [rs.block_fwd_static(x, dw, H, r, want_full=True) for x in xs]     # two calls in a row
    got.append(rs.block_fwd_static(xs[0], dw, H, r, want_full=True))         # stale scratch from call 2
    rs.static_async_status(ctx.device)       # the static kernels' own status word: no bounded wait ran out
    ctx.async_status()
    for g, wnt in zip(got, want + [want[0]]):
        for k in ("x_out", "scores", "keep_idx", "x_full"):
            assert torch.equal(g[k], wnt[k]), k
    with pytest.raises(rs.RsError) as e:
        big = torch.zeros(64, N, D, dtype=tdt, device="cuda")
        rs.block_fwd_static(big, dw, H, r)
    assert e.value.status == 3
    del big
    # The property the entry point exists for: the call itself takes no device memory.  Straight
    # through the C ABI with buffers made beforehand, neither the driver's free-memory figure nor
    # torch's allocator moves across the call.
    from paper_2508_00367_b200 import binding
    lib = binding.load_library()
    x = xs[1]
    K = N - r
    code = binding.RS_BF16 if tdt == torch.bfloat16 else binding.RS_F32
    desc = binding.BlockDesc(code, code, B, N, D, H, dw.D_mlp, r, 1, 0.0, 0.0, 0, 0)
    x_out = torch.empty(B, K, D, dtype=tdt, device="cuda")
    scores = torch.empty(B, N, dtype=torch.float32, device="cuda")
    keep = torch.empty(B, K, dtype=torch.int32, device="cuda")
    err = ctypes.create_string_buffer(256)
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)
    # (Python's collector is kept out of the measured stretch: tensors that earlier tests left in
    # reference cycles would otherwise be returned to torch's allocator in the middle of it.)
    import gc
    gc.collect()
    torch.cuda.synchronize()
    gc.disable()
    try:
        free0, alloc0, reserved0 = torch.cuda.mem_get_info()[0], torch.cuda.memory_allocated(), torch.cuda.memory_reserved()
        st = lib.rs_block_fwd_static(ctypes.byref(desc), ctypes.byref(dw.struct), x.data_ptr(), x_out.data_ptr(),
                                     scores.data_ptr(), keep.data_ptr(), None, stream, err, 256)
        assert st == 0, err.value
        assert lib.rs_static_async_status(stream, err, 256) == 0, err.value
        assert torch.cuda.mem_get_info()[0] == free0
        assert torch.cuda.memory_allocated() == alloc0 and torch.cuda.memory_reserved() == reserved0
    finally:
        gc.enable()
    assert torch.equal(x_out, want[1]["x_out"]) and torch.equal(keep, want[1]["keep_idx"]) and torch.equal(scores, want[1]["scores"])
    ctx.close()
