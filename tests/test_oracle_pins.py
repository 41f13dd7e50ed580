"""Pins for the CPU oracle: every routine in oracle/ is checked against
something that is not itself -- brute force by an independent NumPy routine,
torch-CPU fp64 library routines as special cases, closed forms, invariants,
and the GFLOPs the paper prints.  No GPU."""
import math
import os

import numpy as np
import pytest
import torch

import brute
from oracle import rs_oracle as orc
from oracle import schedule as osched

RNG = np.random.default_rng(1234)
GOLD = os.path.join(os.path.dirname(__file__), "golden")


# ----------------------------------------------------------------- attention (Eq. sa)

@pytest.mark.parametrize("N,d", [(1, 4), (2, 3), (5, 4), (8, 2)])
def test_attn_vs_brute_force(N, d):
    B, H = 2, 3
    q, k, v = (RNG.normal(size=(B, N, H, d)) for _ in range(3))
    got = orc.attn(q, k, v, scale=0.37)
    for b in range(B):
        for h in range(H):
            want = brute.softmax_attention(q[b, :, h], k[b, :, h], v[b, :, h], 0.37)
            np.testing.assert_allclose(got[b, :, h], want, rtol=0, atol=1e-13)


def test_attn_vs_torch_library():
    B, N, H, d = 2, 37, 3, 16
    q, k, v = (RNG.normal(size=(B, N, H, d)) for _ in range(3))
    got = orc.attn(q, k, v)  # default scale 1/sqrt(d)
    tq, tk, tv = (torch.from_numpy(a).permute(0, 2, 1, 3) for a in (q, k, v))
    want = torch.softmax(tq @ tk.transpose(-1, -2) / math.sqrt(d), dim=-1) @ tv
    np.testing.assert_allclose(got, want.permute(0, 2, 1, 3).numpy(), rtol=0, atol=1e-13)


def test_attn_closed_forms():
    B, N, H, d = 1, 6, 2, 4
    q, k, v = (RNG.normal(size=(B, N, H, d)) for _ in range(3))
    # one token: output is its value row
    np.testing.assert_allclose(orc.attn(q[:, :1], k[:, :1], v[:, :1]), v[:, :1], atol=1e-15)
    # zero queries: uniform weights -> column mean of V
    got = orc.attn(np.zeros_like(q), k, v)
    np.testing.assert_allclose(got, np.broadcast_to(v.mean(axis=1, keepdims=True), v.shape), atol=1e-14)
    # all value rows equal: output is that row whatever the logits
    vv = np.broadcast_to(v[:, :1], v.shape).copy()
    np.testing.assert_allclose(orc.attn(q, k, vv), vv, atol=1e-14)
    # one key dominating by a 60-logit margin: output ~ its value row
    k2 = np.zeros_like(k)
    q2 = np.zeros_like(q)
    q2[..., 0] = 1.0
    k2[:, 3, :, 0] = 60.0
    got = orc.attn(q2, k2, v, scale=1.0)
    np.testing.assert_allclose(got, np.broadcast_to(v[:, 3:4], v.shape), atol=1e-12)
    # permuting the tokens permutes the outputs (no positional dependence)
    perm = RNG.permutation(N)
    np.testing.assert_allclose(orc.attn(q[:, perm], k[:, perm], v[:, perm]),
                               orc.attn(q, k, v)[:, perm], atol=1e-14)
    # a transposed operand (q <-> k) must change the answer
    assert np.abs(orc.attn(k, q, v) - orc.attn(q, k, v)).max() > 1e-3
    # heads are independent: changing head 1's keys leaves head 0 alone
    k3 = k.copy()
    k3[:, :, 1] += 1.0
    np.testing.assert_array_equal(orc.attn(q, k3, v)[:, :, 0], orc.attn(q, k, v)[:, :, 0])


def test_attn_softmax_shift_invariance_large_logits():
    # the max-subtraction must make +1000 logits harmless
    B, N, H, d = 1, 5, 1, 2
    q = np.full((B, N, H, d), 100.0)
    k = RNG.normal(size=(B, N, H, d)) + 10.0
    v = RNG.normal(size=(B, N, H, d))
    got = orc.attn(q, k, v, scale=1.0)
    assert np.isfinite(got).all()
    want = brute.softmax_attention(q[0, :, 0], k[0, :, 0], v[0, :, 0], 1.0)
    np.testing.assert_allclose(got[0, :, 0], want, atol=1e-12)


# ----------------------------------------------------------------- LN, linear, GELU

def test_layernorm_vs_torch_and_invariants():
    T, D = 7, 48
    x = RNG.normal(size=(T, D)) * 3 + 1
    g, b = RNG.normal(size=D), RNG.normal(size=D)
    got = orc.layernorm(x, g, b, eps=1e-6)
    want = torch.nn.functional.layer_norm(torch.from_numpy(x), (D,), torch.from_numpy(g),
                                          torch.from_numpy(b), eps=1e-6).numpy()
    np.testing.assert_allclose(got, want, atol=1e-13)
    y = orc.layernorm(x, np.ones(D), np.zeros(D), eps=1e-6)
    np.testing.assert_allclose(y.mean(-1), 0, atol=1e-14)
    var = x.var(-1)
    np.testing.assert_allclose(y.var(-1), var / (var + 1e-6), rtol=1e-12)
    # constant token -> beta
    np.testing.assert_allclose(orc.layernorm(np.full((1, D), 3.3), g, b, 1e-6), b[None], atol=1e-12)
    # eps really is inside the square root
    big = orc.layernorm(x, np.ones(D), np.zeros(D), eps=10.0)
    np.testing.assert_allclose(big.var(-1), var / (var + 10.0), rtol=1e-12)


def test_linear_vs_library_and_layout():
    T, I, O = 5, 11, 7
    x, W, b = RNG.normal(size=(T, I)), RNG.normal(size=(O, I)), RNG.normal(size=O)
    np.testing.assert_allclose(orc.linear(x, W, b), x @ W.T + b, atol=1e-13)
    np.testing.assert_allclose(orc.linear(x, W, None), x @ W.T, atol=1e-13)
    # [out, in] layout: unit weight matrix picks input column `i` into output `o`
    E = np.zeros((O, I))
    E[2, 9] = 1.0
    y = orc.linear(x, E)
    np.testing.assert_allclose(y[:, 2], x[:, 9], atol=0)
    assert np.abs(np.delete(y, 2, axis=1)).max() == 0


def test_gelu_vs_torch_and_closed_forms():
    t = np.linspace(-6, 6, 101)
    want = torch.nn.functional.gelu(torch.from_numpy(t), approximate="none").numpy()
    np.testing.assert_allclose(orc.gelu(t), want, atol=1e-14)
    assert orc.gelu(np.zeros(1))[0] == 0.0
    np.testing.assert_allclose(orc.gelu(np.array([40.0])), [40.0], atol=0)
    np.testing.assert_allclose(orc.gelu(-t), orc.gelu(t) - t, atol=1e-14)  # GELU(-t) = GELU(t) - t
    # the tanh approximation differs by ~1e-3: the oracle must be the erf form
    tanh = torch.nn.functional.gelu(torch.from_numpy(t), approximate="tanh").numpy()
    assert np.abs(orc.gelu(t) - tanh).max() > 1e-4


# ----------------------------------------------------------------- shift score (Sec. 3.2)

def test_shift_score_closed_forms():
    B, N, D = 2, 5, 8
    x = RNG.normal(size=(B, N, D))
    # identity layer -> zero shift
    assert np.all(orc.shift_score(x, x) == 0.0)
    # 3-4-5 triangle
    a = np.zeros((1, 1, D)); a[0, 0, 0], a[0, 0, 1] = 3.0, 4.0
    assert orc.shift_score(a, np.zeros_like(a))[0, 0] == 5.0
    assert orc.shift_score(a, np.zeros_like(a), "l1")[0, 0] == 7.0
    # one coordinate moved by c -> |c|, for both norms
    y = x.copy(); y[1, 2, 3] -= 2.5
    s = orc.shift_score(y, x)
    assert s[1, 2] == 2.5 and np.count_nonzero(s) == 1
    assert orc.shift_score(y, x, "l1")[1, 2] == 2.5
    # homogeneity and symmetry of a norm; independent formula via numpy
    y = RNG.normal(size=(B, N, D))
    np.testing.assert_allclose(orc.shift_score(-3 * y, -3 * x), 3 * orc.shift_score(y, x), rtol=1e-14)
    np.testing.assert_allclose(orc.shift_score(y, x), orc.shift_score(x, y), rtol=0, atol=0)
    np.testing.assert_allclose(orc.shift_score(y, x), np.linalg.norm(y - x, axis=-1), rtol=1e-14)
    np.testing.assert_allclose(orc.shift_score(y, x, "l1"), np.linalg.norm(y - x, ord=1, axis=-1), rtol=1e-14)
    # cosine: parallel 0, opposite 2, orthogonal 1, scale invariant
    e0 = np.zeros((1, 1, D)); e0[..., 0] = 2.0
    e1 = np.zeros((1, 1, D)); e1[..., 1] = 5.0
    assert abs(orc.shift_score(3 * e0, e0, "cos")[0, 0]) < 1e-15
    assert abs(orc.shift_score(-e0, e0, "cos")[0, 0] - 2.0) < 1e-15
    assert abs(orc.shift_score(e1, e0, "cos")[0, 0] - 1.0) < 1e-15
    np.testing.assert_allclose(orc.shift_score(7 * y, x, "cos"), orc.shift_score(y, x, "cos"), atol=1e-14)
    want = 1 - (x * y).sum(-1) / (np.linalg.norm(x, axis=-1) * np.linalg.norm(y, axis=-1))
    np.testing.assert_allclose(orc.shift_score(y, x, "cos"), want, atol=1e-14)


# ----------------------------------------------------------------- selection and compaction

@pytest.mark.parametrize("has_cls", [True, False])
def test_topk_vs_brute_force_with_ties(has_cls):
    for trial in range(60):
        N = int(RNG.integers(1, 13))
        r = int(RNG.integers(0, N))
        s = RNG.integers(0, 4, size=(3, N)).astype(np.float64)  # many ties
        if trial % 5 == 0 and N > 2:
            s[0, RNG.integers(0, N)] = np.nan
            s[1, RNG.integers(0, N)] = np.inf
        got = orc.topk(s, r, has_cls)
        assert got.shape == (3, N - r)
        for b in range(3):
            np.testing.assert_array_equal(got[b], brute.select(list(s[b]), r, has_cls))


def test_topk_invariants():
    B, N = 4, 197
    s = np.abs(RNG.normal(size=(B, N)))
    s[:, 0] = 0.0  # CLS has the lowest score and must survive anyway
    for r in (0, 1, 16, N - 2, N - 1):
        keep = orc.topk(s, r, True)
        assert keep.shape == (B, N - r)
        assert (keep[:, 0] == 0).all()
        assert (np.diff(keep, axis=1) > 0).all() if N - r > 1 else True
        for b in range(B):
            dropped = np.setdiff1d(np.arange(N), keep[b])
            kept_nc = keep[b][keep[b] != 0]
            if len(dropped) and len(kept_nc):
                assert s[b, dropped].max() <= s[b, kept_nc].min()
    np.testing.assert_array_equal(orc.topk(s, 0, True), np.tile(np.arange(N, dtype=np.int32), (B, 1)))
    # without the CLS rule token 0 (score 0) is the first to go
    assert 0 not in orc.topk(s, 1, False)[0]
    # all scores equal -> lowest indices kept
    np.testing.assert_array_equal(orc.topk(np.ones((1, 9)), 4, True)[0], np.arange(5))
    np.testing.assert_array_equal(orc.topk(np.ones((1, 9)), 4, False)[0], np.arange(5))
    # "lowest scores are dropped", not the highest
    np.testing.assert_array_equal(orc.topk(np.array([[9., 1., 5., 3.]]), 2, False)[0], [0, 2])
    with pytest.raises(ValueError):
        orc.topk(s, N, True)
    with pytest.raises(ValueError):
        orc.topk(s, -1, True)


def test_gather_is_row_selection():
    B, N, D = 2, 9, 5
    x = RNG.normal(size=(B, N, D))
    keep = np.array([[0, 2, 8], [1, 3, 4]], dtype=np.int32)
    out = orc.gather(x, keep)
    for b in range(B):
        for j in range(3):
            np.testing.assert_array_equal(out[b, j], x[b, keep[b, j]])


# ----------------------------------------------------------------- the block (Eq. att, Eq. MLP)

def _rand_weights(D, Dm, zero_mlp_out=False):
    w = dict(ln1_g=1 + 0.1 * RNG.normal(size=D), ln1_b=0.1 * RNG.normal(size=D),
             w_qkv=0.2 * RNG.normal(size=(3 * D, D)), b_qkv=0.1 * RNG.normal(size=3 * D),
             w_o=0.2 * RNG.normal(size=(D, D)), b_o=0.1 * RNG.normal(size=D),
             ln2_g=1 + 0.1 * RNG.normal(size=D), ln2_b=0.1 * RNG.normal(size=D),
             w_fc1=0.2 * RNG.normal(size=(Dm, D)), b_fc1=0.1 * RNG.normal(size=Dm),
             w_fc2=0.2 * RNG.normal(size=(D, Dm)), b_fc2=0.1 * RNG.normal(size=D))
    if zero_mlp_out:
        w["w_fc2"][:] = 0
        w["b_fc2"][:] = 0
    return w


def test_block_vs_independent_numpy_block():
    B, N, D, H, Dm, r = 2, 7, 12, 3, 20, 3
    x = RNG.normal(size=(B, N, D))
    w = _rand_weights(D, Dm)
    res = orc.block_fwd(x, w, H, r, has_cls=True, eps=1e-6)
    for b in range(B):
        xp, m, xh = brute.block(x[b], w, H, 1e-6, 1 / math.sqrt(D // H))
        np.testing.assert_allclose(res["x_prime"][b], xp, atol=1e-12)
        np.testing.assert_allclose(res["m"][b], m, atol=1e-12)
        np.testing.assert_allclose(res["x_hat"][b], xh, atol=1e-12)
        s = np.sqrt(((m - xp) ** 2).sum(-1))
        np.testing.assert_allclose(res["scores"][b], s, rtol=1e-12)
        keep = brute.select(list(res["scores"][b]), r, True)
        np.testing.assert_array_equal(res["keep_idx"][b], keep)
        np.testing.assert_array_equal(res["x_out"][b], res["x_hat"][b][keep])


def test_block_score_modes_and_invariants():
    B, N, D, H, Dm, r = 1, 6, 8, 2, 16, 2
    x = RNG.normal(size=(B, N, D))
    w = _rand_weights(D, Dm)
    base = orc.block_fwd(x, w, H, r)
    a = base["x_prime"] - x  # SA(LN(x)) incl. projection
    # (ii) literal: ||MLP(LN(x')) - x'||;  delta reading: ||x^ - x'|| = ||m||
    np.testing.assert_allclose(base["scores"], np.linalg.norm(base["m"] - base["x_prime"], axis=-1), rtol=1e-13)
    np.testing.assert_allclose(orc.block_fwd(x, w, H, r, score_mode="mlp_delta")["scores"],
                               np.linalg.norm(base["m"], axis=-1), rtol=1e-12)
    # (i) ||SA(LN(x)) - x||  and (iii) ||x^ - x||
    np.testing.assert_allclose(orc.block_fwd(x, w, H, r, score_mode="attn")["scores"],
                               np.linalg.norm(a - x, axis=-1), rtol=1e-12)
    np.testing.assert_allclose(orc.block_fwd(x, w, H, r, score_mode="block")["scores"],
                               np.linalg.norm(base["x_hat"] - x, axis=-1), rtol=1e-12)
    # a zero MLP branch gives x^ = x' and a zero "delta" score
    w0 = _rand_weights(D, Dm, zero_mlp_out=True)
    z = orc.block_fwd(x, w0, H, r, score_mode="mlp_delta")
    np.testing.assert_array_equal(z["x_hat"], z["x_prime"])
    assert np.all(z["scores"] == 0)
    # kept count, CLS, order
    assert base["keep_idx"].shape == (B, N - r) and base["keep_idx"][0, 0] == 0
    assert base["x_out"].shape == (B, N - r, D)
    # samples are independent: a batch of two equals two batches of one
    x2 = np.concatenate([x, RNG.normal(size=(1, N, D))])
    both = orc.block_fwd(x2, w, H, r)
    np.testing.assert_allclose(both["x_hat"][0], base["x_hat"][0], atol=1e-14)


def test_model_loop_feeds_rounded_outputs():
    B, N, D, H, Dm = 1, 9, 8, 2, 16
    x = RNG.normal(size=(B, N, D))
    blocks = [_rand_weights(D, Dm) for _ in range(3)]
    outs = orc.model_fwd(x, blocks, H, [2, 0, 3], io_dtype="bf16")
    assert [o["x_out"].shape[1] for o in outs] == [7, 7, 4]
    one = orc.block_fwd(outs[0]["x_out_rounded"], blocks[1], H, 0)
    np.testing.assert_array_equal(one["x_hat"], outs[1]["x_hat"])


# ----------------------------------------------------------------- rounding helpers

def test_round_bf16_matches_torch():
    a = np.concatenate([RNG.normal(size=4096) * 10.0 ** RNG.integers(-6, 6, size=4096),
                        [0.0, -0.0, 1.0, 1.00390625, 1.0078125, 1.01171875, np.inf, -np.inf]])
    want = torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    np.testing.assert_array_equal(orc.round_bf16(a), want)
    assert np.isnan(orc.round_bf16(np.array([np.nan]))[0])


# ----------------------------------------------------------------- schedule and MAC model

def _gold_rows():
    for line in open(os.path.join(GOLD, "gmacs.txt")):
        if line.startswith("#") or not line.strip():
            continue
        f = line.split()
        yield f[0], int(f[1]), int(f[2]), int(f[3]), int(f[4]), int(f[5]), f[6], float(f[7])


def _sched(sch, N0, L):
    if sch == "none":
        return osched.drops_ratio(N0, L, 0.0, [])
    ratio = float(sch[5:sch.index("@")])
    layers = [int(t) for t in sch[sch.index("@") + 1:].split(",")]
    return osched.drops_ratio(N0, L, ratio, layers)


def test_schedule_reproduces_printed_gmacs():
    for name, D, L, N0, pt, pi, sch, printed in _gold_rows():
        Ns, _ = _sched(sch, N0, L)
        got = osched.model_gmacs(Ns, D, pt, pi)
        assert abs(got - printed) <= 0.1 + 1e-9, (name, sch, got, printed)


def test_other_schedule_readings_miss_printed_gmacs():
    # pruning BEFORE the listed block, or 0-based layer numbers, do not give the printed values
    def before(N0, L, ratio, layers):
        N, Ns = N0, []
        for l in range(1, L + 1):
            if l in layers:
                N -= int(math.floor(ratio * N))
            Ns.append(N)
        return Ns
    assert abs(osched.model_gmacs(before(2353, 12, 0.2, [1, 2, 3]), 768, 2352, 768) - 156.4) > 5
    Ns0, _ = osched.drops_ratio(197, 12, 0.2, [2, 5, 8])  # "[1,4,7]" read 0-based, after
    assert abs(osched.model_gmacs(Ns0, 384, 196, 768) - 3.0) > 0.1


def test_fixed_schedule_counts():
    Ns, rs = osched.drops_fixed(197, 12, 16)
    assert Ns == [197 - 16 * i for i in range(12)] and sum(rs) == 192 and Ns[-1] - rs[-1] == 5
    Ns, rs = osched.drops_ratio(1569, 12, 0.30, (3, 6, 9))
    assert Ns[0] == 1569 and Ns[3] == 1099 and Ns[6] == 770 and Ns[9] == 539
    Ns, rs = osched.drops_ratio(4097, 24, 0.25, (4, 8, 12, 16))
    assert [Ns[i] for i in (0, 4, 8, 12, 16)] == [4097, 3073, 2305, 1729, 1297]


# ----------------------------------------------------------------- line-wise pruning of a 2-D grid (Sec. 4, CNN)

def test_linewise_vs_brute_force_with_ties():
    for trial in range(60):
        H, W = int(RNG.integers(1, 8)), int(RNG.integers(1, 8))
        dr, dc = int(RNG.integers(0, H)), int(RNG.integers(0, W))
        s = RNG.integers(0, 3, size=(2, H, W)).astype(np.float64)      # few values: many equal averages
        kr, kc = orc.linewise(s, dr, dc)
        assert kr.shape == (2, H - dr) and kc.shape == (2, W - dc)
        for b in range(2):
            wr, wc = brute.linewise([list(r) for r in s[b]], dr, dc)
            np.testing.assert_array_equal(kr[b], wr)
            np.testing.assert_array_equal(kc[b], wc)


def test_linewise_closed_forms():
    # separable map s[h, w] = a[h] + c[w]: a row's average is a[h] + mean(c), so rows rank by a and
    # columns by c, whatever the other factor is
    a = np.array([5.0, 1.0, 4.0, 2.0, 3.0, 0.5])
    c = np.array([0.25, 9.0, 3.0, 7.0])
    s = (a[:, None] + c[None, :])[None]
    kr, kc = orc.linewise(s, 2, 1)
    np.testing.assert_array_equal(kr[0], [0, 2, 3, 4])     # a = 1.0 and 0.5 go
    np.testing.assert_array_equal(kc[0], [1, 2, 3])        # c = 0.25 goes
    # both averages come from the full grid.  Here the row that goes (average -1) holds the weight of
    # column 1: on the full grid column 0 averages -4/3 and goes; had the row been removed first,
    # column 0 would average 3 against 0 and column 1 would go instead.
    s2 = np.array([[[3.0, 0.0], [3.0, 0.0], [-10.0, 8.0]]])
    kr, kc = orc.linewise(s2, 1, 1)
    np.testing.assert_array_equal(kr[0], [0, 1])
    np.testing.assert_array_equal(kc[0], [1])
    # equal averages: the later line goes
    s3 = np.array([[[0.0, 9.0], [0.0, 9.0], [50.0, 0.0]]])
    np.testing.assert_array_equal(orc.linewise(s3, 1, 0)[0][0], [0, 2])
    # one column: the grid is a token list without a class token
    t = RNG.normal(size=(3, 11))
    np.testing.assert_array_equal(orc.linewise(t[:, :, None], 4, 0)[0], orc.topk(t, 4, False))
    np.testing.assert_array_equal(orc.linewise(t[:, None, :], 0, 4)[1], orc.topk(t, 4, False))
    # transposing the grid swaps the two answers
    g = RNG.normal(size=(2, 6, 9))
    kr, kc = orc.linewise(g, 2, 3)
    kr_t, kc_t = orc.linewise(np.ascontiguousarray(g.transpose(0, 2, 1)), 3, 2)
    np.testing.assert_array_equal(kr, kc_t)
    np.testing.assert_array_equal(kc, kr_t)
    # nothing dropped: identity; dropping everything is refused
    kr, kc = orc.linewise(g, 0, 0)
    np.testing.assert_array_equal(kr[0], np.arange(6))
    np.testing.assert_array_equal(kc[1], np.arange(9))
    with pytest.raises(ValueError):
        orc.linewise(g, 6, 0)
    with pytest.raises(ValueError):
        orc.linewise(g, 0, 9)


def test_grid_gather_is_fancy_indexing():
    x = RNG.normal(size=(2, 5, 7, 3))
    kr = np.array([[0, 2, 4], [1, 2, 3]], dtype=np.int32)
    kc = np.array([[6, 5], [0, 3]], dtype=np.int32)           # any order is taken as given
    got = orc.grid_gather(x, kr, kc)
    for b in range(2):
        np.testing.assert_array_equal(got[b], x[b][kr[b]][:, kc[b]])

