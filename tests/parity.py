"""Shared comparison rules of the GPU parity tests.

Tolerances (from the build's target statement):
  * integer / index / byte work: bit-exact;
  * bf16 storage: max-abs 2e-2 and mean-abs 2e-3 against oracle outputs rounded
    the same way.  A bf16 value with |v| >= 4 has an ulp of 2^-5 > 2e-2, so for
    bf16 *outputs* one rounding flip is allowed: per element max(2e-2, 1 ulp);
    the un-rounded (fp32-out) result is held to the literal 2e-2;
  * fp32 storage: max-abs 1e-4, mean-abs 1e-5 (fp32 FMA arithmetic over K <= 1536
    terms of magnitude <= ~1 gives ~1e-6; the margin covers exp/erf/rsqrt);
  * kept-index sets equal, except tokens whose oracle scores lie within 1e-3
    relative of each other.
"""
import numpy as np

BF16_MAX_ABS, BF16_MEAN_ABS = 2e-2, 2e-3
F32_MAX_ABS, F32_MEAN_ABS = 1e-4, 1e-5
TIE_REL = 1e-3


def bf16_ulp(v):
    a = np.abs(np.asarray(v, dtype=np.float64))
    e = np.floor(np.log2(np.maximum(a, 2.0 ** -126)))
    return 2.0 ** (e - 7)


def check_float(got, want, dtype, rounded_output):
    """got: GPU result (any float array); want: oracle result already rounded the same way."""
    got = np.asarray(got, dtype=np.float64)
    want = np.asarray(want, dtype=np.float64)
    assert got.shape == want.shape, (got.shape, want.shape)
    if got.size == 0:
        return dict(max_abs=0.0, mean_abs=0.0, over=0)
    err = np.abs(got - want)
    assert np.isfinite(got).all(), "non-finite GPU output"
    if dtype == "bf16":
        tol = np.maximum(BF16_MAX_ABS, bf16_ulp(want)) if rounded_output else BF16_MAX_ABS
        mean_tol = BF16_MEAN_ABS
    else:
        tol, mean_tol = F32_MAX_ABS, F32_MEAN_ABS
    over = int((err > BF16_MAX_ABS).sum()) if dtype == "bf16" else 0
    assert (err <= tol).all(), f"max-abs {err.max():.3e} (limit {np.min(tol):.1e}), {int((err > tol).sum())} elements over"
    assert err.mean() <= mean_tol, f"mean-abs {err.mean():.3e} > {mean_tol:.1e}"
    return dict(max_abs=float(err.max()), mean_abs=float(err.mean()), over=over)


def check_keep(oracle_scores, keep_oracle, keep_gpu, has_cls=True):
    """Kept sets must agree except inside a 1e-3-relative score band.  Returns the
    number of samples whose sets differ (tolerated)."""
    keep_oracle = np.asarray(keep_oracle)
    keep_gpu = np.asarray(keep_gpu)
    assert keep_gpu.shape == keep_oracle.shape
    B, K = keep_gpu.shape
    N = oracle_scores.shape[1]
    swaps = 0
    for b in range(B):
        g = keep_gpu[b]
        assert (np.diff(g) > 0).all(), "keep_idx not strictly ascending"
        assert K == 0 or (g[0] >= 0 and g[-1] < N)
        if has_cls and K > 0:
            assert g[0] == 0, "class token dropped"
        so, sg = set(keep_oracle[b].tolist()), set(g.tolist())
        if so == sg:
            continue
        diff = np.array(sorted(so ^ sg))
        s = oracle_scores[b, diff]
        band = s.max() - s.min()
        assert band < TIE_REL * abs(s.max()), f"sample {b}: kept sets differ outside the tie band ({band:.3e} vs {s.max():.3e})"
        swaps += 1
    return swaps
