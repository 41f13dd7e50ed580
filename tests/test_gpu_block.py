"""GPU parity of rs_block_fwd and of the layer loop against the CPU oracle."""
import numpy as np
import pytest
import torch

import parity
from oracle import rs_oracle as orc
from paper_2508_00367_b200 import synth

pytestmark = pytest.mark.gpu

DT = {"f32": torch.float32, "bf16": torch.bfloat16}


@pytest.fixture(scope="module")
def ctx():
    import paper_2508_00367_b200 as rs
    c = rs.Context(0)
    yield c
    c.async_status()
    c.close()


def _np(w):
    return {k: v.double().numpy() for k, v in w.items()}


def _run_block(ctx, x, w, H, r, dtype, out_dtype=None, score_mode="mlp", has_cls=True, dist="l2"):
    import paper_2508_00367_b200 as rs
    dw = rs.DeviceBlockWeights(w, DT[dtype], ctx.device)
    res = ctx.block_fwd(x.to(DT[dtype]).cuda(), dw, H, r, has_cls=has_cls, out_dtype=out_dtype,
                        score_mode=score_mode, want_full=True, dist=dist)
    torch.cuda.synchronize()
    return {k: v.cpu() for k, v in res.items()}


def _check_block(res, ref, dtype, out_dtype, has_cls=True, score_rel=None):
    od = "f32" if out_dtype == torch.float32 else dtype
    rounded = od == "bf16"
    want_full = orc.round_to(ref["x_hat"], od)
    stats = parity.check_float(res["x_full"].double().numpy(), want_full, dtype, rounded)
    s = res["scores"].double().numpy()
    rel = np.abs(s - ref["scores"]) / np.maximum(np.abs(ref["scores"]), 1e-30)
    if score_rel is None:
        score_rel = 1e-5 if dtype == "f32" else 5e-4
    assert rel.max() < score_rel, f"score rel err {rel.max():.3e}"
    swaps = parity.check_keep(ref["scores"], ref["keep_idx"], res["keep_idx"].numpy(), has_cls)
    # compaction is an exact row copy of the GPU's own un-pruned output
    keep = res["keep_idx"].long()
    B = keep.shape[0]
    for b in range(B):
        assert torch.equal(res["x_out"][b], res["x_full"][b][keep[b]])
    return stats, swaps


def test_block_vit_s_fp32_config(ctx):
    wl = synth.WORKLOADS["vit_s_block"]
    x, blocks = synth.make_workload(wl, seed=0)
    ref = orc.block_fwd(x.double().numpy(), _np(blocks[0]), wl.H, wl.drops[0])
    res = _run_block(ctx, x, blocks[0], wl.H, wl.drops[0], "f32")
    assert res["x_out"].shape == (2, 181, 384)
    _check_block(res, ref, "f32", None)


@pytest.mark.parametrize("out_dtype", [None, torch.float32])
@pytest.mark.parametrize("B,N,D,H,r", [(3, 197, 768, 12, 16), (2, 129, 384, 6, 0), (2, 21, 768, 12, 16),
                                       (1, 577, 1024, 16, 20), (2, 64, 128, 2, 63), (1, 1, 64, 1, 0)])
def test_block_bf16(ctx, B, N, D, H, r, out_dtype):
    x = synth.make_tokens(B, N, D, "bf16", seed=N)
    w = synth.make_block_weights(D, 4 * D, "bf16", seed=N + 1)
    ref = orc.block_fwd(x.double().numpy(), _np(w), H, r)
    res = _run_block(ctx, x, w, H, r, "bf16", out_dtype)
    _check_block(res, ref, "bf16", out_dtype)


def test_block_delta_score_mode_and_no_cls(ctx):
    # |x^ - x'| = |MLP(LN(x'))| is ~10x smaller than the default score, so bf16 contraction
    # error is ~1e-3 of it: the kept-set rule is checked in fp32 storage, bf16 gets scores only
    B, N, D, H, r = 2, 100, 384, 6, 30
    x = synth.make_tokens(B, N, D, "f32", seed=5)
    w = synth.make_block_weights(D, 4 * D, "f32", seed=6)
    ref = orc.block_fwd(x.double().numpy(), _np(w), H, r, has_cls=False, score_mode="mlp_delta")
    res = _run_block(ctx, x, w, H, r, "f32", None, score_mode="mlp_delta", has_cls=False)
    _check_block(res, ref, "f32", None, has_cls=False)
    xb = synth.make_tokens(B, N, D, "bf16", seed=5)
    wb = synth.make_block_weights(D, 4 * D, "bf16", seed=6)
    refb = orc.block_fwd(xb.double().numpy(), _np(wb), H, r, has_cls=False, score_mode="mlp_delta")
    resb = _run_block(ctx, xb, wb, H, r, "bf16", torch.float32, score_mode="mlp_delta", has_cls=False)
    rel = np.abs(resb["scores"].double().numpy() - refb["scores"]) / refb["scores"]
    assert rel.max() < 3e-3
    parity.check_float(resb["x_full"].double().numpy(), refb["x_hat"], "bf16", False)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode", ["attn", "block"])
def test_block_other_operation_choices(ctx, dtype, mode):
    """Sec. 3.3 operation choices (i) and (iii): the shift through attention, fused into the
    projection epilogue, and through the whole block, fused into the FC2 epilogue."""
    B, N, D, H, r = 2, 150, 384, 6, 11
    x = synth.make_tokens(B, N, D, dtype, seed=41)
    w = synth.make_block_weights(D, 4 * D, dtype, seed=42)
    ref = orc.block_fwd(x.double().numpy(), _np(w), H, r, score_mode=mode)
    out_dtype = torch.float32 if dtype == "bf16" else None
    res = _run_block(ctx, x, w, H, r, dtype, out_dtype, score_mode=mode)
    # These scores are norms of the sub-layer outputs themselves (no exact x' term dominates them as in
    # the default mode), so they carry the bf16 operand rounding of the contractions in full: 2e-3.
    _check_block(res, ref, dtype, out_dtype, score_rel=(1e-5 if dtype == "f32" else 2e-3))


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("mode,dist", [("mlp", "l1"), ("mlp", "cos"), ("mlp_delta", "cos"), ("attn", "l1"),
                                       ("attn", "cos"), ("block", "cos"), ("block", "l1")])
def test_block_other_distances(ctx, dtype, mode, dist):
    """Sec. 3.3 distance metrics (L1, cosine) fused into the same epilogues as the default L2."""
    B, N, D, H, r = 2, 140, 256, 4, 9
    x = synth.make_tokens(B, N, D, dtype, seed=51)
    w = synth.make_block_weights(D, 4 * D, dtype, seed=52)
    ref = orc.block_fwd(x.double().numpy(), _np(w), H, r, score_mode=mode, dist=dist)
    out_dtype = torch.float32 if dtype == "bf16" else None
    res = _run_block(ctx, x, w, H, r, dtype, out_dtype, score_mode=mode, dist=dist)
    full = res["x_full"].double().numpy()
    parity.check_float(full, orc.round_to(ref["x_hat"], "f32"), dtype, False)
    s = res["scores"].double().numpy()
    if dist == "cos":          # a distance in [0, 2]: absolute tolerance
        tol = 1e-5 if dtype == "f32" else 2e-3
        assert np.abs(s - ref["scores"]).max() < tol, np.abs(s - ref["scores"]).max()
    else:
        rel = np.abs(s - ref["scores"]) / np.maximum(np.abs(ref["scores"]), 1e-30)
        assert rel.max() < (1e-5 if dtype == "f32" else 2e-3), rel.max()
    assert res["keep_idx"].shape == (B, N - r) and (res["keep_idx"][:, 0] == 0).all()
    keep = res["keep_idx"].numpy()
    if dtype == "f32":
        parity.check_keep(ref["scores"], ref["keep_idx"], keep)
    else:
        # bf16 contractions put up to `tol` of error on these scores, more than the 1e-3 tie band: a
        # token may change sides only if its oracle score lies within 2 tol of the oracle's cut
        tol = 2e-3
        for b in range(B):
            assert (np.diff(keep[b]) > 0).all()
            so, sg = set(ref["keep_idx"][b].tolist()), set(keep[b].tolist())
            sb = ref["scores"][b]
            cut = np.sort(sb[1:])[::-1][N - r - 2]          # lowest kept score among the non-CLS tokens
            for t in so ^ sg:
                lim = 2 * tol * (1.0 if dist == "cos" else abs(cut))
                assert abs(sb[t] - cut) <= lim, (b, t, sb[t], cut)


def test_block_video_tokens_ar1(ctx):
    # 4 frames x 49 patches + CLS, temporally correlated tokens, ratio pruning
    B, N, D, H = 2, 197, 768, 12
    x = synth.make_tokens(B, N, D, "bf16", frames=4, seed=9)
    w = synth.make_block_weights(D, 4 * D, "bf16", seed=10)
    r = int(0.3 * N)
    ref = orc.block_fwd(x.double().numpy(), _np(w), H, r)
    res = _run_block(ctx, x, w, H, r, "bf16", torch.float32)
    _check_block(res, ref, "bf16", torch.float32)


def test_block_video_vit_l14_token_count(ctx):
    """One block at the video ViT-L/14 size (16 frames x 256 patches + CLS = 4097 tokens, D = 1024,
    16 heads, 25 % dropped), one sample: the long-sequence attention path (33 key tiles, one CTA per
    item), the radix selection and every GEMM shape of that workload, against the oracle."""
    B, N, D, H = 1, 4097, 1024, 16
    x = synth.make_tokens(B, N, D, "bf16", frames=16, seed=3)
    w = synth.make_block_weights(D, 4 * D, "bf16", seed=4)
    r = N // 4
    ref = orc.block_fwd(x.double().numpy(), _np(w), H, r)
    res = _run_block(ctx, x, w, H, r, "bf16", torch.float32)
    _check_block(res, ref, "bf16", torch.float32)


def test_block_rejects_bad_arguments(ctx):
    import paper_2508_00367_b200 as rs
    x = synth.make_tokens(1, 8, 64, "bf16", seed=1)
    w = synth.make_block_weights(64, 256, "bf16", seed=2)
    dw = rs.DeviceBlockWeights(w, torch.bfloat16, ctx.device)
    with pytest.raises(rs.RsError) as e:
        ctx.block_fwd(x.to(torch.bfloat16).cuda(), dw, 1, 8)              # r = N
    assert e.value.status == 1
    with pytest.raises(rs.RsError) as e:
        ctx.block_fwd(x.to(torch.bfloat16).cuda(), dw, 2, 1)              # head_dim 32
    assert e.value.status == 2
    small = torch.empty(256, dtype=torch.uint8, device="cuda")
    with pytest.raises(rs.RsError) as e:
        ctx.block_fwd(x.to(torch.bfloat16).cuda(), dw, 1, 1, workspace=small)
    assert e.value.status == 3
    ctx.async_status()


@pytest.mark.parametrize("name,nsamp", [("vit_b16", 2), ("vit_l16_384", 1), ("video_vit_b16", 1), ("video_vit_l14", 1)])
def test_model_layer_forced_full_batch(ctx, name, nsamp):
    """Every bf16 workload at its full launch configuration (ViT-B/16: B = 64, 12 blocks, 16 tokens
    dropped per block; ViT-L/16 at 384 px: B = 32, 24 blocks, 20 per block; video ViT-B/16: B = 16,
    1569 tokens, 30 % dropped after blocks 3, 6, 9; video ViT-L/14: B = 4, 4097 tokens, 25 % dropped
    after blocks 4, 8, 12, 16).  The oracle runs the whole model on `nsamp` samples; every block of
    the GPU model is fed the oracle's rounded input for that block, tiled to the full batch, so the
    GEMM tile widths, the attention item list and the selection grid are those of the benchmark, and a
    tolerated tie swap in one block cannot leak into the next.  Outputs, scores and kept sets of
    every block are compared (Eq. att, Eq. MLP, Sec. 3.1 / 3.2)."""
    import paper_2508_00367_b200 as rs
    wl = synth.WORKLOADS[name]
    x, blocks = synth.make_workload(wl, seed=0, B=nsamp)
    outs = orc.model_fwd(x.double().numpy(), [_np(w) for w in blocks], wl.H, list(wl.drops), io_dtype="bf16")
    cur = orc.round_bf16(x.double().numpy())
    total_swaps, worst = 0, dict(max_abs=0.0, mean_abs=0.0, over=0)
    for l, w in enumerate(blocks):
        dw = rs.DeviceBlockWeights(w, torch.bfloat16, ctx.device)
        xin = torch.from_numpy(cur).to(torch.bfloat16).repeat(wl.B // nsamp, 1, 1).cuda()
        assert xin.shape == (wl.B, outs[l]["scores"].shape[1], wl.D)
        res = ctx.block_fwd(xin, dw, wl.H, wl.drops[l], want_full=True)
        torch.cuda.synchronize()
        res = {k: v.cpu() for k, v in res.items()}
        for k in res:   # every copy of the samples gives identical results
            assert torch.equal(res[k][:nsamp], res[k][-nsamp:]), k
        first = {k: v[:nsamp] for k, v in res.items()}
        stats, swaps = _check_block(first, outs[l], "bf16", None)
        total_swaps += swaps
        worst = {k: max(worst[k], stats[k]) for k in worst}
        cur = outs[l]["x_out_rounded"]
        del dw, xin, res
    ctx.async_status()
    print(f"{name}: tolerated tie swaps over {wl.L} blocks x {nsamp} samples: {total_swaps}; worst block {worst}")


def test_model_free_running_matches_until_first_swap(ctx):
    """The layer loop (PrunedViT) against the oracle's own free run, 4 blocks of the
    ViT-B/16 workload, B = 2: outputs must agree block by block for as long as the kept
    sets are identical."""
    import paper_2508_00367_b200 as rs
    wl = synth.WORKLOADS["vit_b16"]
    x, blocks = synth.make_workload(wl, seed=1, B=2, L=4)
    drops = list(wl.drops[:4])
    outs = orc.model_fwd(x.double().numpy(), [_np(w) for w in blocks], wl.H, drops, io_dtype="bf16")
    model = rs.PrunedViT(ctx, blocks, wl.H, drops, torch.bfloat16)
    got = model.forward(x.to(torch.bfloat16).cuda())
    torch.cuda.synchronize()
    alive = [True, True]
    compared = 0
    for l in range(4):
        for b in range(2):
            if not alive[b]:
                continue
            if not np.array_equal(got[l]["keep_idx"][b].cpu().numpy(), outs[l]["keep_idx"][b]):
                parity.check_keep(outs[l]["scores"][b:b + 1], outs[l]["keep_idx"][b:b + 1],
                                  got[l]["keep_idx"][b:b + 1].cpu().numpy())
                alive[b] = False
                continue
            g = got[l]["x_out"][b].cpu().double().numpy()
            want = outs[l]["x_out_rounded"][b]
            err = np.abs(g - want)
            # free run: one-ulp rounding flips of earlier blocks ride along the residual stream
            # (the layer-forced test above is the parity check proper), so this is a drift
            # bound: the literal mean for the first block, 2.5x that later, a loose cap per element
            assert err.mean() <= (parity.BF16_MEAN_ABS if l == 0 else 2.5 * parity.BF16_MEAN_ABS)
            assert err.max() <= 0.125   # a handful of elements sit several ulps off by block 4
            compared += 1
    assert compared >= 2


def test_graph_replay_equals_eager(ctx):
    """PrunedViT.forward(graph=True) replays the same kernels: outputs are bit-identical to the
    eager loop, on a first and on a repeated replay."""
    import paper_2508_00367_b200 as rs
    from paper_2508_00367_b200 import synth
    B, N, D, H, L = 3, 150, 256, 4, 3
    x = synth.make_tokens(B, N, D, "bf16", seed=5).to(torch.bfloat16).cuda()
    blocks = [synth.make_block_weights(D, 4 * D, "bf16", seed=10 + l) for l in range(L)]
    model = rs.PrunedViT(ctx, blocks, H, [10, 0, 7], torch.bfloat16)
    eager = [{k: v.clone() for k, v in o.items()} for o in model.forward(x)]
    for _ in range(2):
        outs = model.forward(x, graph=True)
        torch.cuda.synchronize()
        for a, b in zip(eager, outs):
            assert torch.equal(a["keep_idx"], b["keep_idx"])
            assert torch.equal(a["x_out"].view(torch.int16), b["x_out"].view(torch.int16))
            assert torch.equal(a["scores"], b["scores"])
    # seven kernels up to the FC2 epilogue, then two for a block that drops tokens (ranking, rows) or one
    # (scores and identity indices) for a tapped block that drops none; the block after a pruning block
    # gets its LN1 from that block's row kernel and launches none: blocks 0 and 2 -> 9, block 1 -> 7
    assert model.launches_per_forward(B, N, D) == 9 + 7 + 9
    ctx.async_status()


@pytest.mark.parametrize("B,N,D,H,drops,dt", [
    (2, 197, 384, 6, [16, 0, 20, 5], "bf16"),
    (1, 1100, 128, 2, [76, 0, 30], "bf16"),        # N > 1024: radix selection and the stand-alone gather kernel
    (2, 50, 128, 2, [5, 5, 0], "f32"),             # fp32 storage (SIMT kernels)
])
def test_vit_fwd_equals_the_block_loop(ctx, B, N, D, H, drops, dt):
    """rs_vit_fwd / rs_vit_fwd_taps are the layer loop inside the library.  They fold LN1 of the block
    after a pruning block into the compaction kernel (same row arithmetic), so every block's outputs
    are bit-identical to chaining rs_block_fwd."""
    import paper_2508_00367_b200 as rs
    from paper_2508_00367_b200 import synth
    tdt = torch.bfloat16 if dt == "bf16" else torch.float32
    x = synth.make_tokens(B, N, D, dt, seed=61).to(tdt).cuda()
    blocks = [synth.make_block_weights(D, 4 * D, dt, seed=70 + l) for l in range(len(drops))]
    model = rs.PrunedViT(ctx, blocks, H, drops, tdt)
    chain, cur = [], x
    for l, r in enumerate(drops):
        o = ctx.block_fwd(cur, model.weights[l], H, r)
        chain.append(o)
        cur = o["x_out"]
    taps = model.forward(x)                                      # rs_vit_fwd_taps: every block's outputs
    torch.cuda.synchronize()
    for want, got_l in zip(chain, taps):
        assert torch.equal(got_l["keep_idx"], want["keep_idx"])
        assert torch.equal(got_l["scores"], want["scores"])
        assert torch.equal(got_l["x_out"], want["x_out"])
    # outputs requested for some blocks only: the others' tokens stay in the two workspace buffers
    some = ctx.vit_fwd_taps(x, model.weights, H, drops, tap_blocks=[1])
    torch.cuda.synchronize()
    assert sorted(some) == sorted({1, len(drops) - 1})
    for l, got_l in some.items():
        assert torch.equal(got_l["keep_idx"], chain[l]["keep_idx"])
        assert torch.equal(got_l["scores"], chain[l]["scores"])
        assert torch.equal(got_l["x_out"], chain[l]["x_out"])
    want = chain[-1]
    got = ctx.vit_fwd(x, model.weights, H, drops)
    torch.cuda.synchronize()
    assert torch.equal(got["keep_idx"], want["keep_idx"])
    assert torch.equal(got["scores"], want["scores"])
    assert torch.equal(got["x_out"], want["x_out"])
    with pytest.raises(rs.RsError):
        ctx.vit_fwd(x, model.weights, H, drops[:-1] + [N])       # the last block cannot drop all its tokens
    ctx.async_status()


@pytest.mark.parametrize("mode,dist", [("block", "l2"), ("attn", "cos"), ("mlp_delta", "l1")])
def test_vit_fwd_in_place_pruning_other_scores(ctx, mode, dist):
    """A pruning block whose compacted tokens nobody asks for writes no dense copy: the next block
    reads the kept rows of the un-pruned output through the index list (LN1, the projection's
    residual and, for the whole-block shift, the FC2 epilogue's second residual).  Same bits as
    chaining rs_block_fwd, for the operation choices and distances of Sec. 3.3 that read the block
    input in an epilogue."""
    import paper_2508_00367_b200 as rs
    B, N, D, H, drops = 3, 333, 256, 4, [40, 33, 0, 50, 7]
    x = synth.make_tokens(B, N, D, "bf16", seed=81).to(torch.bfloat16).cuda()
    blocks = [synth.make_block_weights(D, 4 * D, "bf16", seed=90 + l) for l in range(len(drops))]
    weights = [rs.DeviceBlockWeights(w, torch.bfloat16, ctx.device) for w in blocks]
    chain, cur = [], x
    for l, r in enumerate(drops):
        o = ctx.block_fwd(cur, weights[l], H, r, score_mode=mode, dist=dist)
        chain.append(o)
        cur = o["x_out"]
    got = ctx.vit_fwd(x, weights, H, drops, score_mode=mode, dist=dist)          # only the last block is materialised
    some = ctx.vit_fwd_taps(x, weights, H, drops, tap_blocks=[2], score_mode=mode, dist=dist)
    torch.cuda.synchronize()
    for k in ("x_out", "scores", "keep_idx"):
        assert torch.equal(got[k], chain[-1][k]), k
        assert torch.equal(some[2][k], chain[2][k]), k
        assert torch.equal(some[4][k], chain[4][k]), k
    ctx.async_status()


def test_tensor_maps_are_encoded_once_per_buffer():
    """A repeated block call on the same buffers encodes no tensor map again (the context keeps them per
    pointer, shape and box; a fresh context, so that its 128 slots are not yet contended), and gives
    the same bits."""
    import paper_2508_00367_b200 as rs
    ctx = rs.Context(0)
    B, N, D, H, r = 2, 150, 256, 4, 10
    x = synth.make_tokens(B, N, D, "bf16", seed=3).to(torch.bfloat16).cuda()
    w = synth.make_block_weights(D, 4 * D, "bf16", seed=4)
    dw = rs.DeviceBlockWeights(w, torch.bfloat16, ctx.device)
    desc = ctx.block_desc(B, N, D, H, dw.D_mlp, r, torch.bfloat16)
    ws = torch.empty(ctx.block_workspace_bytes(desc), dtype=torch.uint8, device="cuda")
    bufs = dict(x_out=torch.empty(B, N - r, D, dtype=torch.bfloat16, device="cuda"),
                scores=torch.empty(B, N, dtype=torch.float32, device="cuda"),
                keep_idx=torch.empty(B, N - r, dtype=torch.int32, device="cuda"))
    first = {k: v.clone() for k, v in ctx.block_fwd(x, dw, H, r, workspace=ws, **bufs).items()}
    h0, m0 = ctx.tmap_cache_stats()
    again = ctx.block_fwd(x, dw, H, r, workspace=ws, **bufs)
    h1, m1 = ctx.tmap_cache_stats()
    torch.cuda.synchronize()
    assert m1 == m0 and h1 > h0, (h0, m0, h1, m1)
    for k in first:
        assert torch.equal(first[k], again[k]), k
    ctx.async_status()
    ctx.close()


@pytest.mark.parametrize("B,N,D,H,drops", [(3, 197, 256, 4, [0, 0, 16]), (2, 300, 512, 8, [0, 40, 0, 0]),
                                           (64, 197, 768, 12, [0, 0])])
def test_layer_loop_with_ln1_folded_into_qkv(ctx, B, N, D, H, drops):
    """rs_prepare_ln1_fold: a block whose predecessor drops nothing runs no LN1 kernel, its QKV product reads
    the tokens themselves and normalises in its epilogue from the sums the previous FC2 left.  Every block
    of the folded loop against the oracle fed that block's actual input (Eq. att, Eq. MLP, Sec. 3.2 / 3.1),
    and one launch less per folded block."""
    import paper_2508_00367_b200 as rs
    L = len(drops)
    x = synth.make_tokens(B, N, D, "bf16", seed=3 * N + D)
    blocks = [synth.make_block_weights(D, 4 * D, "bf16", seed=50 + l) for l in range(L)]
    plain = rs.PrunedViT(ctx, blocks, H, drops, torch.bfloat16)
    folded = rs.PrunedViT(ctx, blocks, H, drops, torch.bfloat16, fold_ln1=True)
    dx = x.to(torch.bfloat16).cuda()
    n0 = ctx.launch_count()
    outs_p = [{k: v.clone() for k, v in o.items()} for o in plain.forward(dx)]
    n1 = ctx.launch_count()
    outs = [{k: v.cpu() for k, v in o.items()} for o in folded.forward(dx)]
    n2 = ctx.launch_count()
    ctx.async_status()
    n_folded = sum(1 for l in range(1, L) if drops[l - 1] == 0)
    assert (n1 - n0) - (n2 - n1) == n_folded
    cur = x.to(torch.bfloat16)
    nsamp = min(B, 2)                       # the oracle on the first samples; the batch exercises the tiling
    for l in range(L):
        ref = orc.block_fwd(cur[:nsamp].double().numpy(), _np(blocks[l]), H, drops[l])
        o = outs[l]
        sc = o["scores"][:nsamp].double().numpy()
        rel = np.abs(sc - ref["scores"]) / np.maximum(np.abs(ref["scores"]), 1e-30)
        assert rel.max() < 5e-4, (l, rel.max())
        parity.check_keep(ref["scores"], ref["keep_idx"], o["keep_idx"][:nsamp].numpy(), True)
        for b in range(nsamp):
            want = orc.round_to(ref["x_hat"][b][o["keep_idx"][b].long().numpy()], "bf16")
            parity.check_float(o["x_out"][b].double().numpy()[None], want[None], "bf16", True)
        # the folded loop stays within rounding of the plain one
        torch.testing.assert_close(o["x_out"].float(), outs_p[l]["x_out"].cpu().float(), rtol=4e-2, atol=4e-2)
        cur = o["x_out"]

