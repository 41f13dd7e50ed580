"""Independent NumPy restatement of the path's definitions, used only to pin
the C oracle.  Written from the equations with explicit loops where the index
order matters; shares nothing with oracle/ or with the CUDA package."""
import math

import numpy as np


def softmax_attention(q, k, v, scale):
    """Eq. sa for one head: q, k, v [N, d]."""
    N = q.shape[0]
    out = np.zeros_like(v, dtype=np.float64)
    for i in range(N):
        logits = np.array([scale * float(np.dot(q[i], k[j])) for j in range(N)])
        w = np.exp(logits - logits.max())
        w = w / w.sum()
        for j in range(N):
            out[i] += w[j] * v[j]
    return out


def layer_norm(x, g, b, eps):
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * g + b


def gelu(t):
    return np.vectorize(lambda z: 0.5 * z * (1.0 + math.erf(z / math.sqrt(2.0))))(t)


def block(x, w, H, eps, scale):
    """x [N, D] one sample -> (x_prime, m, x_hat) by Eq. att and Eq. MLP."""
    N, D = x.shape
    dh = D // H
    u = layer_norm(x, w["ln1_g"], w["ln1_b"], eps)
    qkv = u @ w["w_qkv"].T + w["b_qkv"]
    o = np.zeros((N, D))
    for h in range(H):
        sl = slice(h * dh, (h + 1) * dh)
        o[:, sl] = softmax_attention(qkv[:, sl], qkv[:, D + h * dh:D + (h + 1) * dh],
                                     qkv[:, 2 * D + h * dh:2 * D + (h + 1) * dh], scale)
    x_prime = o @ w["w_o"].T + w["b_o"] + x
    u2 = layer_norm(x_prime, w["ln2_g"], w["ln2_b"], eps)
    m = gelu(u2 @ w["w_fc1"].T + w["b_fc1"]) @ w["w_fc2"].T + w["b_fc2"]
    return x_prime, m, m + x_prime


def select(scores, r, has_cls):
    """Keep the N - r best of one sample: higher score first, lower index on a
    tie, NaN last, token 0 first when has_cls.  Selection by repeated removal
    of the worst token -- deliberately not a sort."""
    alive = list(range(len(scores)))

    def worse(i, j):  # True if i ranks below j
        if has_cls and (i == 0 or j == 0):
            return j == 0
        si, sj = scores[i], scores[j]
        if math.isnan(si) or math.isnan(sj):
            if math.isnan(si) and math.isnan(sj):
                return i > j
            return math.isnan(si)
        if si != sj:
            return si < sj
        return i > j

    for _ in range(r):
        w = alive[0]
        for i in alive[1:]:
            if worse(i, w):
                w = i
        alive.remove(w)
    return np.array(sorted(alive), dtype=np.int32)


def linewise(scores, drop_rows, drop_cols):
    """Line-wise pruning of one H x W grid of scores, from the definition: the average of every
    row and of every column (exact rational arithmetic, so no summation order enters), then the
    lines with the lowest averages go, by the same ranking as tokens (no pinned line)."""
    from fractions import Fraction
    H, W = len(scores), len(scores[0])

    def avg(vals):
        if any(math.isnan(v) or math.isinf(v) for v in vals):
            return float(sum(vals)) / len(vals)
        return float(sum(Fraction(v) for v in vals) / len(vals))

    rows = [avg([scores[h][w] for w in range(W)]) for h in range(H)]
    cols = [avg([scores[h][w] for h in range(H)]) for w in range(W)]
    return select(rows, drop_rows, False), select(cols, drop_cols, False)

