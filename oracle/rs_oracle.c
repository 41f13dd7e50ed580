/*
 * rs_oracle.c -- TEST INFRASTRUCTURE, NOT PRODUCT CODE.
 *
 * A plain, slow, fp64 CPU statement of what the Representation Shift hot path
 * computes: one pre-LN Vision-Transformer block (Eq. att, Eq. MLP), the
 * representation-shift score of Sec. 3.2 (s = D(F(x), x)), and the removal of
 * the r lowest-score tokens (Sec. 3.1, "reduced token set"), plus the line-wise
 * pruning of a 2-D token grid (Sec. 4, CNN).  Only the tests,
 * the smoke check and the benchmark's cpu_baseline / reference arm may call
 * it.  It shares no code with the CUDA library and includes none of its
 * headers.
 *
 * Every routine is the textbook definition written as loops.  There is no
 * blocking, fusion or reordering; the attention matrix is materialised per
 * (sample, head) because that is the definition the fused GPU kernel must
 * reproduce (Eq. sa).  OpenMP only spreads independent rows / samples over
 * cores; it does not change any sum's order.
 *
 * Pins (tests/test_oracle_pins.py): brute force on tiny inputs by an
 * independent NumPy routine, torch-CPU fp64 library routines (softmax,
 * layer_norm, gelu, matmul) as special cases, closed forms and invariants.
 * Whole-block numerics have no value printed in the paper to compare with:
 * "parity unpinned" by the paper for orc_block_fwd as a whole; it is pinned by
 * the composition of its pinned parts and by agreement with the independent
 * NumPy brute-force block.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

int orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

/* LN in Eq. att / Eq. MLP: per token, mean and biased variance over the D
 * features, then affine.  out may not alias x. */
void orc_layernorm(const double* x, const double* gamma, const double* beta, double eps,
                   long T, int D, double* out) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        const double* xr = x + t * (long)D;
        double mu = 0.0;
        for (int c = 0; c < D; ++c) mu += xr[c];
        mu /= (double)D;
        double var = 0.0;
        for (int c = 0; c < D; ++c) var += (xr[c] - mu) * (xr[c] - mu);
        var /= (double)D;
        double rstd = 1.0 / sqrt(var + eps);
        for (int c = 0; c < D; ++c) out[t * (long)D + c] = (xr[c] - mu) * rstd * gamma[c] + beta[c];
    }
}

/* y[t, o] = bias[o] + sum_i x[t, i] * W[o, i], i ascending.  W is [out, in]
 * (the transpose of the paper's W in "[Q,K,V] = xW").  bias may be NULL.  W is
 * first copied into [in, out] order so the inner loop runs over contiguous
 * outputs; every output still adds its terms in the order i = 0, 1, ... */
void orc_linear(const double* x, const double* W, const double* bias, long T, int in, int out,
                double* y) {
    double* Wt = (double*)malloc(sizeof(double) * (size_t)in * (size_t)out);
    for (int o = 0; o < out; ++o)
        for (int i = 0; i < in; ++i) Wt[(long)i * out + o] = W[(long)o * in + i];
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        const double* xr = x + t * (long)in;
        double* yr = y + t * (long)out;
        for (int o = 0; o < out; ++o) yr[o] = bias ? bias[o] : 0.0;
        for (int i = 0; i < in; ++i) {
            const double xi = xr[i];
            const double* wr = Wt + (long)i * out;
            for (int o = 0; o < out; ++o) yr[o] += xi * wr[o];
        }
    }
    free(Wt);
}

/* Exact GELU: t * Phi(t), Phi the standard normal CDF. */
void orc_gelu(double* x, long n) {
#pragma omp parallel for schedule(static)
    for (long i = 0; i < n; ++i) x[i] = x[i] * 0.5 * (1.0 + erf(x[i] / sqrt(2.0)));
}

/* Eq. sa per (sample, head): S = q k^T * scale, P = row softmax(S), o = P v.
 * q, k, v, out: contiguous [B, N, H, dh].  The N x N matrix is written out in
 * full on purpose. */
void orc_attn(const double* q, const double* k, const double* v, int B, int N, int H, int dh,
              double scale, double* out) {
#pragma omp parallel for collapse(2) schedule(dynamic)
    for (int b = 0; b < B; ++b) {
        for (int h = 0; h < H; ++h) {
            double* S = (double*)malloc(sizeof(double) * (size_t)N * (size_t)N);
            long rs = (long)H * dh; /* row stride */
            const double* qb = q + ((long)b * N) * rs + (long)h * dh;
            const double* kb = k + ((long)b * N) * rs + (long)h * dh;
            const double* vb = v + ((long)b * N) * rs + (long)h * dh;
            double* ob = out + ((long)b * N) * rs + (long)h * dh;
            for (int i = 0; i < N; ++i)
                for (int j = 0; j < N; ++j) {
                    double acc = 0.0;
                    for (int c = 0; c < dh; ++c) acc += qb[i * rs + c] * kb[j * rs + c];
                    S[(long)i * N + j] = acc * scale;
                }
            for (int i = 0; i < N; ++i) {
                double* Si = S + (long)i * N;
                double mx = Si[0];
                for (int j = 1; j < N; ++j) mx = Si[j] > mx ? Si[j] : mx;
                double den = 0.0;
                for (int j = 0; j < N; ++j) { Si[j] = exp(Si[j] - mx); den += Si[j]; }
                for (int j = 0; j < N; ++j) Si[j] /= den;
            }
            for (int i = 0; i < N; ++i) {
                for (int c = 0; c < dh; ++c) ob[i * rs + c] = 0.0;
                for (int j = 0; j < N; ++j) {
                    const double p = S[(long)i * N + j];
                    for (int c = 0; c < dh; ++c) ob[i * rs + c] += p * vb[j * rs + c];
                }
            }
            free(S);
        }
    }
}

/* Sec. 3.2 / "Distance metrics": per token t, s[t] = D(after[t,:], before[t,:]).
 * dist 0: L2 norm of the difference; 1: L1 norm; 2: cosine distance
 * 1 - <a,b>/(|a||b|), denominator floored at 1e-12 (the paper gives no rule
 * for zero vectors). */
void orc_shift_score(const double* after, const double* before, long T, int D, int dist,
                     double* s) {
#pragma omp parallel for schedule(static)
    for (long t = 0; t < T; ++t) {
        const double* a = after + t * (long)D;
        const double* b = before + t * (long)D;
        if (dist == 0) {
            double acc = 0.0;
            for (int c = 0; c < D; ++c) acc += (a[c] - b[c]) * (a[c] - b[c]);
            s[t] = sqrt(acc);
        } else if (dist == 1) {
            double acc = 0.0;
            for (int c = 0; c < D; ++c) acc += fabs(a[c] - b[c]);
            s[t] = acc;
        } else {
            double ab = 0.0, aa = 0.0, bb = 0.0;
            for (int c = 0; c < D; ++c) { ab += a[c] * b[c]; aa += a[c] * a[c]; bb += b[c] * b[c]; }
            double den = sqrt(aa) * sqrt(bb);
            if (den < 1e-12) den = 1e-12;
            s[t] = 1.0 - ab / den;
        }
    }
}

/* Ranking used by the selection: token i outranks token j when its score is
 * larger, or equal with i < j.  NaN ranks below every number.  With has_cls,
 * token 0 outranks everything. */
typedef struct { double s; int idx; int pinned; } orc_tok;

static int orc_rank_cmp(const void* pa, const void* pb) {
    const orc_tok* a = (const orc_tok*)pa;
    const orc_tok* b = (const orc_tok*)pb;
    if (a->pinned != b->pinned) return a->pinned ? -1 : 1;
    int an = isnan(a->s), bn = isnan(b->s);
    if (an != bn) return an ? 1 : -1;
    if (!an) {
        if (a->s > b->s) return -1;
        if (a->s < b->s) return 1;
    }
    return (a->idx > b->idx) - (a->idx < b->idx);
}

static int orc_int_cmp(const void* pa, const void* pb) {
    int a = *(const int32_t*)pa, b = *(const int32_t*)pb;
    return (a > b) - (a < b);
}

/* Sec. 3.2: the r lowest-score tokens are removed, i.e. keep the K = N - r
 * top-ranked tokens of every sample, listed in ascending index.  Returns 0, or
 * -1 for r outside [0, N-1]. */
int orc_topk(const double* scores, int B, int N, int r, int has_cls, int32_t* keep_idx) {
    if (r < 0 || r > N - 1) return -1;
    int K = N - r;
    for (int b = 0; b < B; ++b) {
        orc_tok* tok = (orc_tok*)malloc(sizeof(orc_tok) * (size_t)N);
        for (int i = 0; i < N; ++i) {
            tok[i].s = scores[(long)b * N + i];
            tok[i].idx = i;
            tok[i].pinned = (has_cls && i == 0);
        }
        qsort(tok, (size_t)N, sizeof(orc_tok), orc_rank_cmp);
        int32_t* kb = keep_idx + (long)b * K;
        for (int j = 0; j < K; ++j) kb[j] = tok[j].idx;
        qsort(kb, (size_t)K, sizeof(int32_t), orc_int_cmp);
        free(tok);
    }
    return 0;
}

/* Reduced token set: x_out[b, j, :] = x[b, keep_idx[b, j], :]. */
void orc_gather(const double* x, const int32_t* keep_idx, int B, int N, int K, int D,
                double* x_out) {
    for (int b = 0; b < B; ++b)
        for (int j = 0; j < K; ++j)
            memcpy(x_out + ((long)b * K + j) * D, x + ((long)b * N + keep_idx[(long)b * K + j]) * D,
                   sizeof(double) * (size_t)D);
}

/* Line-wise pruning of a 2-D token grid (Sec. 4, "CNN and SSM", variant L-W): the shift is
 * averaged over every row and over every column of the H x W grid, and the drop_rows rows and
 * drop_cols columns with the lowest averages go, whole lines at a time.  Both averages are taken
 * over the full grid (the text orders neither before the other); a line's rank among its peers
 * follows the token rule (larger average first, lower index on a tie, NaN last).
 * scores [B,H,W]; keep_rows [B,H-drop_rows], keep_cols [B,W-drop_cols], ascending.
 * Returns 0, or -1 when a drop count is outside [0, lines-1]. */
int orc_linewise(const double* scores, int B, int H, int W, int drop_rows, int drop_cols,
                 int32_t* keep_rows, int32_t* keep_cols) {
    if (drop_rows < 0 || drop_rows > H - 1 || drop_cols < 0 || drop_cols > W - 1) return -1;
    double* rm = (double*)malloc(sizeof(double) * (size_t)B * H);
    double* cm = (double*)malloc(sizeof(double) * (size_t)B * W);
    for (int b = 0; b < B; ++b) {
        const double* s = scores + (long)b * H * W;
        for (int h = 0; h < H; ++h) {
            double acc = 0.0;
            for (int w = 0; w < W; ++w) acc += s[(long)h * W + w];
            rm[(long)b * H + h] = acc / (double)W;
        }
        for (int w = 0; w < W; ++w) {
            double acc = 0.0;
            for (int h = 0; h < H; ++h) acc += s[(long)h * W + w];
            cm[(long)b * W + w] = acc / (double)H;
        }
    }
    int rc = orc_topk(rm, B, H, drop_rows, 0, keep_rows);
    if (rc == 0) rc = orc_topk(cm, B, W, drop_cols, 0, keep_cols);
    free(cm); free(rm);
    return rc;
}

/* The grid that is left: x_out[b, i, j, :] = x[b, keep_rows[b, i], keep_cols[b, j], :].
 * x [B,H,W,D] (channels last: a position is a token), x_out [B,Hk,Wk,D]. */
void orc_grid_gather(const double* x, const int32_t* keep_rows, const int32_t* keep_cols, int B, int H, int W,
                     int Hk, int Wk, int D, double* x_out) {
    for (int b = 0; b < B; ++b)
        for (int i = 0; i < Hk; ++i)
            for (int j = 0; j < Wk; ++j)
                memcpy(x_out + (((long)b * Hk + i) * Wk + j) * D,
                       x + (((long)b * H + keep_rows[(long)b * Hk + i]) * W + keep_cols[(long)b * Wk + j]) * D,
                       sizeof(double) * (size_t)D);
}

/* One block followed by pruning.
 *   x' = SA(LN(x)) + x            (Eq. att;  SA includes the output projection)
 *   m  = MLP(LN(x'))              (Eq. MLP without the residual)
 *   x^ = m + x'
 *   score_mode 0: s = ||m - x'||  (operation choice (ii), literal formula)
 *   score_mode 1: s = ||x^ - x'|| = ||m||  (the figure caption's reading of the MLP shift, residual included)
 *   score_mode 2: s = D(SA(LN(x)), x)      (operation choice (i))
 *   score_mode 3: s = D(x^, x)             (operation choice (iii))
 * Outputs (any may be NULL except x_hat): x_prime, m, x_hat [B,N,D]; scores
 * [B,N]; keep_idx [B,N-r]; x_out [B,N-r,D].  Returns 0 or -1 on bad r. */
int orc_block_fwd(const double* x, int B, int N, int D, int H, int Dm,
                  const double* ln1_g, const double* ln1_b,
                  const double* w_qkv, const double* b_qkv,
                  const double* w_o, const double* b_o,
                  const double* ln2_g, const double* ln2_b,
                  const double* w_fc1, const double* b_fc1,
                  const double* w_fc2, const double* b_fc2,
                  double eps, double scale, int score_mode, int dist, int r, int has_cls,
                  double* x_prime, double* m_out, double* x_hat, double* scores,
                  int32_t* keep_idx, double* x_out) {
    if (r < 0 || r > N - 1) return -1;
    long T = (long)B * N;
    int dh = D / H;
    double* u = (double*)malloc(sizeof(double) * T * D);
    double* qkv = (double*)malloc(sizeof(double) * T * 3 * D);
    double* q = (double*)malloc(sizeof(double) * T * D);
    double* k = (double*)malloc(sizeof(double) * T * D);
    double* v = (double*)malloc(sizeof(double) * T * D);
    double* o = (double*)malloc(sizeof(double) * T * D);
    double* a = (double*)malloc(sizeof(double) * T * D);
    double* xp = (double*)malloc(sizeof(double) * T * D);
    double* hid = (double*)malloc(sizeof(double) * T * Dm);
    double* m = (double*)malloc(sizeof(double) * T * D);
    double* s = (double*)malloc(sizeof(double) * T);

    orc_layernorm(x, ln1_g, ln1_b, eps, T, D, u);
    orc_linear(u, w_qkv, b_qkv, T, D, 3 * D, qkv);
    for (long t = 0; t < T; ++t)
        for (int c = 0; c < D; ++c) {
            q[t * D + c] = qkv[t * 3 * D + c];
            k[t * D + c] = qkv[t * 3 * D + D + c];
            v[t * D + c] = qkv[t * 3 * D + 2 * D + c];
        }
    orc_attn(q, k, v, B, N, H, dh, scale, o);
    orc_linear(o, w_o, b_o, T, D, D, a);
    for (long i = 0; i < T * D; ++i) xp[i] = a[i] + x[i];
    orc_layernorm(xp, ln2_g, ln2_b, eps, T, D, u);
    orc_linear(u, w_fc1, b_fc1, T, D, Dm, hid);
    orc_gelu(hid, T * Dm);
    orc_linear(hid, w_fc2, b_fc2, T, Dm, D, m);
    for (long i = 0; i < T * D; ++i) x_hat[i] = m[i] + xp[i];

    if (score_mode == 0) orc_shift_score(m, xp, T, D, dist, s);
    else if (score_mode == 1) orc_shift_score(x_hat, xp, T, D, dist, s);
    else if (score_mode == 2) orc_shift_score(a, x, T, D, dist, s);
    else orc_shift_score(x_hat, x, T, D, dist, s);

    int rc = 0;
    int K = N - r;
    int32_t* keep = (int32_t*)malloc(sizeof(int32_t) * (size_t)B * K);
    rc = orc_topk(s, B, N, r, has_cls, keep);
    if (rc == 0 && x_out) orc_gather(x_hat, keep, B, N, K, D, x_out);
    if (keep_idx) memcpy(keep_idx, keep, sizeof(int32_t) * (size_t)B * K);
    if (scores) memcpy(scores, s, sizeof(double) * T);
    if (x_prime) memcpy(x_prime, xp, sizeof(double) * T * D);
    if (m_out) memcpy(m_out, m, sizeof(double) * T * D);

    free(keep); free(s); free(m); free(hid); free(xp); free(a); free(o);
    free(v); free(k); free(q); free(qkv); free(u);
    return rc;
}
