"""Per-sample token counts (padded layout): every sample of a batch has its own number of tokens and
drops its own number of them.  Each sample is compared with the CPU oracle run on that sample alone
(Eq. sa, Eq. att, Eq. MLP, Sec. 3.1 / 3.2 on its own rows), through the C ABI."""
import numpy as np
import pytest
import torch

import parity
from oracle import rs_oracle as orc
from paper_2508_00367_b200 import synth

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def ctx():
    import paper_2508_00367_b200 as rs
    c = rs.Context(0)
    yield c
    c.async_status()
    c.close()


def _i32(v):
    return torch.tensor(v, dtype=torch.int32, device="cuda")


@pytest.mark.parametrize("N,H,lens", [(197, 3, [197, 1, 64, 65, 128, 129]), (100, 2, [100, 37, 1]),
                                      (700, 2, [700, 513, 129, 300, 5])])
def test_attn_ragged_per_sample_lengths(ctx, N, H, lens):
    B = len(lens)
    g = torch.Generator().manual_seed(N)
    qkv = torch.randn(B, N, 3, H, 64, generator=g).to(torch.bfloat16)
    dq = qkv.cuda()
    out = ctx.attn_fwd_ragged(dq[:, :, 0], dq[:, :, 1], dq[:, :, 2], _i32(lens)).cpu()
    assert torch.isfinite(out.float()).all()
    f = qkv.double().numpy()
    for b, n in enumerate(lens):
        want = orc.attn(f[b:b + 1, :n, 0], f[b:b + 1, :n, 1], f[b:b + 1, :n, 2]).reshape(n, H * 64)
        parity.check_float(out[b, :n].double().numpy(), orc.round_to(want, "bf16"), "bf16", rounded_output=True)
    # the same call with every length = N is the dense entry point, bit for bit, when the dense call runs the
    # kernel that takes per-sample lengths (the dense entry point may pick the other kernel for a shape)
    import os
    import paper_2508_00367_b200 as rs
    os.environ["RS_ATTN_KERNEL"] = "2"
    try:
        two = rs.Context(0)
    finally:
        del os.environ["RS_ATTN_KERNEL"]
    full = two.attn_fwd_ragged(dq[:, :, 0], dq[:, :, 1], dq[:, :, 2], _i32([N] * B))
    assert torch.equal(full, two.attn_fwd(dq[:, :, 0], dq[:, :, 1], dq[:, :, 2]))
    two.async_status()
    two.close()


@pytest.mark.parametrize("N,D,dtype", [(197, 64, torch.bfloat16), (600, 32, torch.float32), (1500, 8, torch.float32)])
def test_topk_compact_ragged_bit_exact(ctx, N, D, dtype):
    rng = np.random.default_rng(N)
    B = 7
    lens = [N, 1, 2, N // 2, N - 1, 65, 64][:B]
    drops = [0, 0, 1, N // 4, N - 2, 64, 10]
    K_pad = N
    s = np.abs(rng.normal(size=(B, N)) * 3 + 10).astype(np.float32)
    s[3, : N // 2 : 3] = 7.0                                     # ties
    x = torch.randn(B, N, D, generator=torch.Generator().manual_seed(1)).to(dtype)
    for has_cls in (True, False):
        xo, keep, lens_out = ctx.topk_compact_ragged(torch.from_numpy(s).cuda(), x.cuda(), _i32(lens), _i32(drops), K_pad, has_cls)
        xo, keep, lens_out = xo.cpu(), keep.cpu().numpy(), lens_out.cpu().numpy()
        for b in range(B):
            n = lens[b]
            r = min(drops[b], n - 1)
            k = n - r
            assert lens_out[b] == k
            want = orc.topk(s[b:b + 1, :n].astype(np.float64), r, has_cls)[0]
            np.testing.assert_array_equal(keep[b, :k], want, err_msg=f"sample {b}")
            assert (keep[b, k:] == -1).all()
            assert torch.equal(xo[b, :k], x[b][torch.from_numpy(want).long()])
            assert (xo[b, k:] == 0).all()


def test_block_ragged_matches_the_oracle_per_sample(ctx):
    """One block on a padded batch of six samples with 40 ... 333 tokens; every sample against the oracle
    on its own rows (outputs, scores, kept indices), padding rows of the output zero."""
    import paper_2508_00367_b200 as rs
    N, D, H = 333, 256, 4
    lens = [333, 40, 129, 257, 64, 200]
    drops = [33, 7, 0, 100, 63, 41]
    B = len(lens)
    K_pad = N                                    # row stride of the outputs: no common minimum drop assumed
    x = synth.make_tokens(B, N, D, "bf16", seed=77)
    for b, n in enumerate(lens):
        x[b, n:] = 0                             # padding rows must be finite: zeros
    w = synth.make_block_weights(D, 4 * D, "bf16", seed=78)
    dw = rs.DeviceBlockWeights(w, torch.bfloat16, ctx.device)
    res = ctx.block_fwd_ragged(x.to(torch.bfloat16).cuda(), dw, H, _i32(lens), _i32(drops), K_pad,
                               out_dtype=torch.float32, want_full=True)
    torch.cuda.synchronize()
    res = {k: v.cpu() for k, v in res.items()}
    wn = {k: v.double().numpy() for k, v in w.items()}
    for b, n in enumerate(lens):
        r = drops[b]
        k = n - r
        ref = orc.block_fwd(x[b:b + 1, :n].double().numpy(), wn, H, r)
        assert int(res["lens_out"][b]) == k
        parity.check_float(res["x_full"][b, :n].double().numpy()[None], ref["x_hat"], "bf16", False)
        sc = res["scores"][b, :n].double().numpy()
        rel = np.abs(sc - ref["scores"][0]) / np.maximum(ref["scores"][0], 1e-30)
        assert rel.max() < 5e-4, (b, rel.max())
        parity.check_keep(ref["scores"], ref["keep_idx"], res["keep_idx"][b:b + 1, :k].numpy())
        kept = res["keep_idx"][b, :k].long()
        assert torch.equal(res["x_out"][b, :k], res["x_full"][b][kept])
        assert (res["x_out"][b, k:] == 0).all() and (res["keep_idx"][b, k:] == -1).all()
    ctx.async_status()


def test_vit_fwd_ragged_equals_the_chain_of_ragged_blocks(ctx):
    """rs_vit_fwd_ragged is rs_block_fwd_ragged chained inside the library: the same bits as chaining the
    calls (each of which is compared with the oracle above), and the counts add up."""
    import paper_2508_00367_b200 as rs
    N, D, H, L = 300, 256, 4, 3
    lens = [300, 41, 129, 257, 180]
    B = len(lens)
    drops = [[30, 5, 10, 64, 20], [20, 0, 40, 33, 100], [0, 35, 9, 60, 7]]      # [L][B]
    pad = [min(d) for d in drops]                                               # 5, 0, 0: the padded length 300 -> 295
    x = synth.make_tokens(B, N, D, "bf16", seed=91)
    for b, n in enumerate(lens):
        x[b, n:] = 0
    dws = [rs.DeviceBlockWeights(synth.make_block_weights(D, 4 * D, "bf16", seed=92 + l), torch.bfloat16, ctx.device)
           for l in range(L)]
    dx = x.to(torch.bfloat16).cuda()
    got = ctx.vit_fwd_ragged(dx, dws, H, pad, _i32(lens), _i32(drops))
    cur, cur_lens, n = dx, _i32(lens), N
    for l in range(L):
        step = ctx.block_fwd_ragged(cur, dws[l], H, cur_lens, _i32(drops[l]), n - pad[l])
        cur, cur_lens, n = step["x_out"], step["lens_out"], n - pad[l]
    assert torch.equal(got["x_out"], cur) and torch.equal(got["keep_idx"], step["keep_idx"])
    assert torch.equal(got["lens_out"], cur_lens)
    want = [max(ln - drops[0][b], 1) for b, ln in enumerate(lens)]
    for l in (1, 2):
        want = [max(w - min(drops[l][b], w - 1), 1) for b, w in enumerate(want)]
    assert got["lens_out"].cpu().tolist() == want
    for b, k in enumerate(want):
        assert (got["x_out"][b, k:] == 0).all() and (got["keep_idx"][b, k:] == -1).all()
        assert torch.isfinite(got["x_out"][b, :k].float()).all() and got["x_out"][b, :k].float().abs().sum() > 0
    ctx.async_status()


def test_ragged_rejects_what_it_cannot_run(ctx):
    import paper_2508_00367_b200 as rs
    q = torch.zeros(1, 8, 1, 64, device="cuda")                  # fp32: no tensor-core kernel
    with pytest.raises(rs.RsError) as e:
        ctx.attn_fwd_ragged(q, q, q, _i32([8]))
    assert e.value.status == 2
    s = torch.zeros(1, 5000, device="cuda")
    with pytest.raises(rs.RsError) as e:
        ctx.topk_compact_ragged(s, None, _i32([5000]), _i32([1]), 5000)
    assert e.value.status == 2
    ctx.async_status()
