"""GPU parity of the three standalone entry points (rs_shift_score,
rs_topk_compact, rs_attn_fwd) against the CPU oracle, through the C ABI."""
import numpy as np
import pytest
import torch

import parity
from oracle import rs_oracle as orc

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2508_00367_b200 as rs
    c = rs.Context(0)
    yield c
    c.async_status()
    c.close()


def _tok(shape, dtype, seed, scale=1.0):
    g = torch.Generator().manual_seed(seed)
    t = torch.randn(*shape, generator=g) * scale
    return t.to(dtype)


DT = {"f32": torch.float32, "bf16": torch.bfloat16}


# ------------------------------------------------------------------ rs_shift_score
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("dist", ["l2", "l1", "cos"])
@pytest.mark.parametrize("B,N,D", [(2, 197, 384), (3, 129, 768), (1, 1, 64), (2, 17, 1024), (1, 5, 8), (1, 3, 2056)])
def test_shift_score(ctx, dtype, dist, B, N, D):
    a = _tok((B, N, D), DT[dtype], 1)
    b = _tok((B, N, D), DT[dtype], 2)
    got = ctx.shift_score(a.cuda(), b.cuda(), dist).cpu().numpy().astype(np.float64)
    want = orc.shift_score(a.double().numpy(), b.double().numpy(), dist)
    if dist == "cos":
        np.testing.assert_allclose(got, want, rtol=0, atol=2e-6)
    else:
        np.testing.assert_allclose(got, want, rtol=2e-6, atol=0)


def test_shift_score_identity_and_empty(ctx):
    a = _tok((2, 33, 768), torch.bfloat16, 3).cuda()
    assert (ctx.shift_score(a, a) == 0).all()
    e = torch.empty(0, 7, 64, dtype=torch.float32, device="cuda")
    assert ctx.shift_score(e, e).shape == (0, 7)


def test_shift_score_full_size(ctx):
    # ViT-B/16 workload, first block: B=64, N=197, D=768 bf16; oracle on sampled tokens
    B, N, D = 64, 197, 768
    a, b = _tok((B, N, D), torch.bfloat16, 4), _tok((B, N, D), torch.bfloat16, 5)
    got = ctx.shift_score(a.cuda(), b.cuda()).cpu().numpy().astype(np.float64)
    idx = np.random.default_rng(0).integers(0, B * N, size=512)
    af, bf = a.double().numpy().reshape(-1, 1, D)[idx], b.double().numpy().reshape(-1, 1, D)[idx]
    np.testing.assert_allclose(got.reshape(-1)[idx], orc.shift_score(af, bf)[:, 0], rtol=2e-6)


# ------------------------------------------------------------------ rs_topk_compact
def _scores(B, N, kind, seed):
    rng = np.random.default_rng(seed)
    if kind == "normal":
        s = np.abs(rng.normal(size=(B, N)) * 5 + 20)
    elif kind == "ties":
        s = rng.integers(0, 5, size=(B, N)).astype(np.float64)
    elif kind == "signed":
        s = rng.normal(size=(B, N))
        s[rng.random((B, N)) < 0.1] = 0.0
        s[rng.random((B, N)) < 0.05] = -0.0
    elif kind == "special":
        s = rng.normal(size=(B, N))
        m = rng.random((B, N))
        s[m < 0.1] = np.nan
        s[(m >= 0.1) & (m < 0.15)] = np.inf
        s[(m >= 0.15) & (m < 0.2)] = -np.inf
    elif kind == "equal":
        s = np.full((B, N), 3.25)
    return s.astype(np.float32)


@pytest.mark.parametrize("kind", ["normal", "ties", "signed", "special", "equal"])
@pytest.mark.parametrize("N", [1, 2, 17, 127, 128, 129, 197, 208, 257, 513, 1024, 1025, 1569, 4097])
def test_topk_compact_bit_exact(ctx, kind, N):
    B, D = 3, 64
    s = _scores(B, N, kind, N)
    x = _tok((B, N, D), torch.bfloat16, N + 1)
    for has_cls in (True, False):
        for r in sorted({0, 1, min(16, N - 1), max(N - 2, 0), N - 1, N // 2}):
            if r > N - 1:
                continue
            xo, keep = ctx.topk_compact(torch.from_numpy(s).cuda(), x.cuda(), r, has_cls)
            want = orc.topk(s.astype(np.float64), r, has_cls)
            np.testing.assert_array_equal(keep.cpu().numpy(), want, err_msg=f"N={N} r={r} cls={has_cls}")
            ref = torch.stack([x[b][torch.from_numpy(want[b]).long()] for b in range(B)])
            assert torch.equal(xo.cpu().view(torch.int16), ref.view(torch.int16))


@pytest.mark.parametrize("kind", ["normal", "ties", "special"])
def test_topk_compact_longest_sequence(ctx, kind):
    # the largest token count the selection takes (the radix kernel's keys fill its shared memory)
    B, N, D = 2, 32768, 8
    s = _scores(B, N, kind, 5)
    x = _tok((B, N, D), torch.float32, 6)
    for r in (1, N // 3, N - 1):
        xo, keep = ctx.topk_compact(torch.from_numpy(s).cuda(), x.cuda(), r, True)
        want = orc.topk(s.astype(np.float64), r, True)
        np.testing.assert_array_equal(keep.cpu().numpy(), want, err_msg=f"r={r}")
        ref = torch.stack([x[b][torch.from_numpy(want[b]).long()] for b in range(B)])
        assert torch.equal(xo.cpu(), ref)


def test_attn_is_reproducible_bit_for_bit(pinned):
    # the same call twice, each kernel: no result depends on the order in which CTAs or warps finish
    qkv = _tok((3, 700, 3, 5, 64), torch.bfloat16, 17).cuda()
    for c in pinned.values():
        a = c.attn_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2])
        b = c.attn_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2])
        assert torch.equal(a, b)


@pytest.mark.parametrize("dtype,D", [("f32", 384), ("bf16", 768), ("bf16", 1024), ("f32", 8)])
def test_topk_compact_rows(ctx, dtype, D):
    B, N, r = 5, 197, 16
    s = _scores(B, N, "normal", 7)
    x = _tok((B, N, D), DT[dtype], 8)
    xo, keep = ctx.topk_compact(torch.from_numpy(s).cuda(), x.cuda(), r, True)
    want = orc.topk(s.astype(np.float64), r, True)
    np.testing.assert_array_equal(keep.cpu().numpy(), want)
    gathered = orc.gather(x.double().numpy(), want)
    np.testing.assert_array_equal(xo.cpu().double().numpy(), gathered)


def test_topk_compact_full_size_and_guard_bands(ctx):
    # video workload shape: B=4, N=4097, D=1024 bf16, 25 % dropped; canaries around the outputs
    B, N, D = 4, 4097, 1024
    r = N // 4
    K = N - r
    s = _scores(B, N, "normal", 11)
    x = _tok((B, N, D), torch.bfloat16, 12)
    pad = 64
    xo_buf = torch.full((B * K * D + 2 * pad,), -7.0, dtype=torch.bfloat16, device="cuda")
    ki_buf = torch.full((B * K + 2 * pad,), -77, dtype=torch.int32, device="cuda")
    xo = xo_buf[pad:pad + B * K * D].view(B, K, D)
    ki = ki_buf[pad:pad + B * K].view(B, K)
    ctx.topk_compact(torch.from_numpy(s).cuda(), x.cuda(), r, True, x_out=xo, keep_idx=ki)
    want = orc.topk(s.astype(np.float64), r, True)
    np.testing.assert_array_equal(ki.cpu().numpy(), want)
    for b in (0, B - 1):
        ref = x[b][torch.from_numpy(want[b]).long()]
        assert torch.equal(xo[b].cpu().view(torch.int16), ref.view(torch.int16))
    assert (xo_buf[:pad] == -7).all() and (xo_buf[-pad:] == -7).all()
    assert (ki_buf[:pad] == -77).all() and (ki_buf[-pad:] == -77).all()


def test_topk_compact_batch_larger_than_the_flag_scratch(ctx):
    """Tokens are ranked by one kernel and moved by another, with a byte per token (and a count per 64
    tokens) in between; a batch with more tokens than that scratch holds (1 MiB)
    runs in several passes."""
    B, N, D, r = 2100, 520, 8, 100
    s = _scores(B, N, "ties", 21)
    x = _tok((B, N, D), torch.float32, 22)
    xo, keep = ctx.topk_compact(torch.from_numpy(s).cuda(), x.cuda(), r, True)
    want = orc.topk(s.astype(np.float64), r, True)
    np.testing.assert_array_equal(keep.cpu().numpy(), want)
    per_sample = 4 * ((N + 63) // 64) + (N + 3) // 4 * 4
    cut = (1 << 20) // per_sample                        # samples that fit one pass
    assert 1 < cut < B
    for b in (0, 1, cut - 1, cut, cut + 1, B - 1):       # both sides of the pass boundary
        assert torch.equal(xo[b].cpu(), x[b][torch.from_numpy(want[b]).long()])
    _, keep2 = ctx.topk_compact(torch.from_numpy(s).cuda(), None, r, False)          # indices only
    np.testing.assert_array_equal(keep2.cpu().numpy(), orc.topk(s.astype(np.float64), r, False))


def test_topk_indices_only_and_errors(ctx):
    s = torch.from_numpy(_scores(2, 50, "normal", 1)).cuda()
    _, keep = ctx.topk_compact(s, None, 10, True)
    np.testing.assert_array_equal(keep.cpu().numpy(), orc.topk(s.cpu().double().numpy(), 10, True))
    import paper_2508_00367_b200 as rs
    with pytest.raises(rs.RsError):
        ctx.topk_compact(s, None, 50, True)          # r > N-1
    with pytest.raises(rs.RsError):
        ctx.topk_compact(s, None, -1, True)
    x = torch.zeros(2, 50, 12, device="cuda")        # D not a multiple of 8
    with pytest.raises(rs.RsError):
        ctx.topk_compact(s, x, 3, True)
    ctx.async_status()                               # context still healthy


# ------------------------------------------------------------------ rs_linewise_compact (Sec. 4, CNN variant L-W)
@pytest.mark.parametrize("kind", ["normal", "ties", "special"])
@pytest.mark.parametrize("B,H,W,D,dr,dc,dtype", [
    (2, 56, 56, 64, 8, 8, "bf16"),        # ResNet stage 1 of a 224 x 224 image: 8 rows and 8 columns go
    (3, 28, 28, 128, 4, 4, "bf16"),       # stage 2: 4 and 4
    (2, 7, 13, 8, 6, 12, "f32"),          # one row and one column left
    (1, 1, 1, 8, 0, 0, "f32"),
    (2, 33, 5, 264, 0, 2, "bf16"),        # ragged channel count (33 pieces of 16 bytes), nothing from the rows
    (1, 256, 256, 8, 100, 3, "bf16"),     # the largest grid
])
def test_linewise_compact_bit_exact(ctx, kind, B, H, W, D, dr, dc, dtype):
    s = _scores(B, H * W, kind, H * 1000 + W).reshape(B, H, W)
    x = _tok((B, H, W, D), DT[dtype], H + W)
    xo, kr, kc = ctx.linewise_compact(torch.from_numpy(s).cuda(), x.cuda(), dr, dc)
    want_r, want_c = orc.linewise(s.astype(np.float64), dr, dc)
    np.testing.assert_array_equal(kr.cpu().numpy(), want_r)
    np.testing.assert_array_equal(kc.cpu().numpy(), want_c)
    want_x = orc.grid_gather(x.double().numpy(), want_r, want_c)
    np.testing.assert_array_equal(xo.cpu().double().numpy(), want_x)


def test_linewise_after_shift_score_and_errors(ctx):
    # the whole step on a feature map: shift of every position across a stage, then the line-wise cut.
    # The oracle ranks the same fp32 scores (the decision is taken on what the score kernel wrote).
    B, H, W, D = 2, 28, 28, 128
    before = _tok((B, H, W, D), torch.bfloat16, 5)
    after = _tok((B, H, W, D), torch.bfloat16, 6)
    sc = ctx.shift_score(after.cuda().view(B, H * W, D), before.cuda().view(B, H * W, D)).view(B, H, W)
    _, kr, kc = ctx.linewise_compact(sc, None, 4, 4)
    want_r, want_c = orc.linewise(sc.cpu().double().numpy(), 4, 4)
    np.testing.assert_array_equal(kr.cpu().numpy(), want_r)
    np.testing.assert_array_equal(kc.cpu().numpy(), want_c)
    full = orc.shift_score(after.double().numpy().reshape(B, H * W, D), before.double().numpy().reshape(B, H * W, D))
    np.testing.assert_allclose(sc.cpu().numpy().reshape(B, H * W).astype(np.float64), full, rtol=2e-6, atol=0)
    import paper_2508_00367_b200 as rs
    for bad in ((H, 0), (0, W), (-1, 0)):
        with pytest.raises(rs.RsError):
            ctx.linewise_compact(sc, None, *bad)
    with pytest.raises(rs.RsError):
        ctx.linewise_compact(torch.zeros(1, 257, 4, device="cuda"), None, 1, 1)       # more lines than supported
    with pytest.raises(rs.RsError):
        ctx.linewise_compact(sc, torch.zeros(B, H, W, 12, device="cuda"), 1, 1)      # D not a multiple of 8
    ctx.async_status()


# ------------------------------------------------------------------ rs_attn_fwd
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("B,N,H", [(2, 197, 6), (1, 1, 1), (1, 2, 2), (2, 17, 3), (1, 127, 2), (1, 128, 2),
                                   (1, 129, 2), (1, 257, 2), (1, 577, 4), (1, 1099, 1)])
def test_attn_packed_qkv(ctx, dtype, B, N, H):
    D = H * 64
    qkv = _tok((B, N, 3, H, 64), DT[dtype], N * 7 + H)
    dq = qkv.cuda()
    got = ctx.attn_fwd(dq[:, :, 0], dq[:, :, 1], dq[:, :, 2]).cpu().double().numpy()
    f = qkv.double().numpy()
    want = orc.attn(f[:, :, 0], f[:, :, 1], f[:, :, 2]).reshape(B, N, D)
    parity.check_float(got, orc.round_to(want, dtype), dtype, rounded_output=True)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_attn_separate_buffers_scale_and_large_logits(ctx, dtype):
    B, N, H = 2, 150, 2
    q = _tok((B, N, H, 64), DT[dtype], 1, scale=3.0)
    k = _tok((B, N, H, 64), DT[dtype], 2, scale=3.0)   # logits of order +-70: needs the max subtraction
    v = _tok((B, N, H, 64), DT[dtype], 3)
    got = ctx.attn_fwd(q.cuda(), k.cuda(), v.cuda(), scale=0.2).cpu().double().numpy()
    want = orc.attn(q.double().numpy(), k.double().numpy(), v.double().numpy(), scale=0.2).reshape(B, N, H * 64)
    parity.check_float(got, orc.round_to(want, dtype), dtype, rounded_output=True)


def test_attn_full_size_video_shape_sampled(ctx):
    # video ViT-L/14 token count (16 x 256 + 1), two heads of one sample; the oracle on sampled query rows
    B, N, H = 1, 4097, 2
    qkv = _tok((B, N, 3, H, 64), torch.bfloat16, 99)
    dq = qkv.cuda()
    got = ctx.attn_fwd(dq[:, :, 0], dq[:, :, 1], dq[:, :, 2]).cpu().double().numpy()
    f = qkv.double().numpy()
    rows = np.unique(np.concatenate([np.arange(0, 3), np.arange(126, 131), np.arange(N - 3, N),
                                     np.random.default_rng(1).integers(0, N, 48)]))
    want = orc.attn(f[:, :, 0], f[:, :, 1], f[:, :, 2]).reshape(B, N, H * 64)[:, rows]
    parity.check_float(got[:, rows], orc.round_to(want, "bf16"), "bf16", rounded_output=True)


@pytest.fixture(scope="module")
def pinned():
    """A context per attention kernel: RS_ATTN_KERNEL is read when the context is made."""
    import os
    import paper_2508_00367_b200 as rs
    made = {}
    for kernel in (2, 3):
        os.environ["RS_ATTN_KERNEL"] = str(kernel)
        try:
            made[kernel] = rs.Context(0)
        finally:
            del os.environ["RS_ATTN_KERNEL"]
    yield made
    for c in made.values():
        c.async_status()
        c.close()


# Both attention kernels on every shape either takes: two query tiles per CTA (kernel 2) and three with
# 64-key tiles (kernel 3).  Token counts around the tile edges (128 rows, 64 keys, groups of three tiles);
# the last two batches are large enough that the leftover tiles of the heads go to the CTAs which the
# last round of groups left out, two to some of them (170 heads), or take turns over all CTAs (200).
@pytest.mark.parametrize("kernel", [2, 3])
@pytest.mark.parametrize("B,N,H", [(1, 129, 2), (1, 192, 1), (1, 193, 1), (1, 257, 2), (2, 384, 3), (1, 385, 2),
                                   (1, 513, 4), (1, 577, 4), (1, 1099, 1), (10, 513, 17), (8, 513, 25)])
def test_attn_each_kernel_pinned(pinned, kernel, B, N, H):
    qkv = _tok((B, N, 3, H, 64), torch.bfloat16, N * 11 + H)
    dq = qkv.cuda()
    got = pinned[kernel].attn_fwd(dq[:, :, 0], dq[:, :, 1], dq[:, :, 2]).cpu().double().numpy()
    f = qkv.double().numpy()
    want = orc.attn(f[:, :, 0], f[:, :, 1], f[:, :, 2]).reshape(B, N, H * 64)
    parity.check_float(got, orc.round_to(want, "bf16"), "bf16", rounded_output=True)


@pytest.mark.parametrize("kernel", [2, 3])
def test_attn_each_kernel_full_size_video_shape_sampled(pinned, kernel):
    B, N, H = 1, 4097, 2
    qkv = _tok((B, N, 3, H, 64), torch.bfloat16, 99)
    dq = qkv.cuda()
    got = pinned[kernel].attn_fwd(dq[:, :, 0], dq[:, :, 1], dq[:, :, 2]).cpu().double().numpy()
    f = qkv.double().numpy()
    rows = np.unique(np.concatenate([np.arange(0, 3), np.arange(126, 131), np.arange(382, 387), np.arange(N - 3, N),
                                     np.random.default_rng(2).integers(0, N, 48)]))
    want = orc.attn(f[:, :, 0], f[:, :, 1], f[:, :, 2]).reshape(B, N, H * 64)[:, rows]
    parity.check_float(got[:, rows], orc.round_to(want, "bf16"), "bf16", rounded_output=True)


def test_launch_log_and_nvtx_ranges_change_nothing(ctx, capfd):
    """RS_LOG=1 prints one line per kernel launch on stderr and RS_NVTX=1 wraps each launch call in a
    range (both are host-side and read when the context is made); the results are the same bits."""
    import os
    import paper_2508_00367_b200 as rs
    os.environ["RS_LOG"] = "1"
    os.environ["RS_NVTX"] = "1"
    try:
        noisy = rs.Context(0)
    finally:
        del os.environ["RS_LOG"], os.environ["RS_NVTX"]
    qkv = _tok((2, 300, 3, 2, 64), torch.bfloat16, 5).cuda()
    a, b = _tok((3, 50, 64), torch.bfloat16, 6).cuda(), _tok((3, 50, 64), torch.bfloat16, 7).cuda()
    capfd.readouterr()
    n0 = noisy.launch_count()
    got = noisy.attn_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2])
    sc = noisy.shift_score(a, b)
    noisy.async_status()
    lines = [ln for ln in capfd.readouterr().err.splitlines() if ln.startswith("rs: launch ")]
    assert len(lines) == noisy.launch_count() - n0 == 2 and all(ln.endswith("-> ok") for ln in lines), lines
    assert torch.equal(got, ctx.attn_fwd(qkv[:, :, 0], qkv[:, :, 1], qkv[:, :, 2]))
    assert torch.equal(sc, ctx.shift_score(a, b))
    noisy.close()


def test_attn_rejects_bad_arguments(ctx):
    import paper_2508_00367_b200 as rs
    q = torch.zeros(1, 4, 2, 32, device="cuda")
    with pytest.raises(rs.RsError) as e:
        ctx.attn_fwd(q, q, q)
    assert e.value.status == 2
    ctx.async_status()


# ------------------------------------------------------------------ rs_linear_fwd
@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("epilogue", ["bias", "gelu", "residual"])
@pytest.mark.parametrize("M,N,K", [(128, 128, 64), (394, 1152, 384), (1000, 768, 3072), (64, 256, 128),
                                   (12608, 768, 768), (77, 2304, 768), (5, 64, 64), (300, 4096, 1024)])
def test_linear(ctx, dtype, epilogue, M, N, K):
    if dtype == "f32" and M * N * K > 4e8:
        pytest.skip("fp32 FMA path: small shapes only")
    a = _tok((M, K), DT[dtype], 1)
    w = _tok((N, K), DT[dtype], 2, scale=0.05)
    b = _tok((N,), torch.float32, 3, scale=0.1)
    res = _tok((M, N), DT[dtype], 4) if epilogue == "residual" else None
    got = ctx.linear_fwd(a.cuda(), w.cuda(), b.cuda(), epilogue, None if res is None else res.cuda())
    got = got.cpu().double().numpy()
    rows = np.arange(M) if M <= 512 else np.unique(np.concatenate(
        [np.arange(0, 130), np.arange(M - 130, M), np.random.default_rng(0).integers(0, M, 64)]))
    want = orc.linear(a.double().numpy()[rows], w.double().numpy(), b.double().numpy())
    if epilogue == "gelu":
        want = orc.gelu(want)
    if epilogue == "residual":
        want = want + res.double().numpy()[rows]
        parity.check_float(got[rows], want, dtype, rounded_output=False)
    else:
        parity.check_float(got[rows], orc.round_to(want, dtype), dtype, rounded_output=True)
