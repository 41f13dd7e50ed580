/*
 * rs.h -- C ABI of the Representation Shift hot path on NVIDIA B200 (sm_100a).
 *
 * The library runs one pre-LN Vision-Transformer block with training-free
 * token pruning:
 *     x'  = SA(LN(x)) + x                      (Eq. att)
 *     x^  = MLP(LN(x')) + x'                   (Eq. MLP)
 *     s_i = D(MLP(LN(x'))_i, x'_i)             (Sec. 3.2, operation choice (ii), D = L2)
 *     x~  = x^ without its r lowest-score tokens   (Sec. 3.1, reduced token set)
 * with an attention kernel that never writes the N x N attention map.
 *
 * Conventions for every entry point
 *   - "dev" pointers are CUDA device pointers owned by the caller; the library
 *     never allocates or frees device memory after rs_create.  Host pointers
 *     are marked "host".
 *   - Tensors are row-major with the innermost dimension contiguous.  Linear
 *     weights are [out, in] (the transpose of the paper's W in "[Q,K,V] = xW").
 *   - Device pointers must be 16-byte aligned; D % 8 == 0; head_dim == 64.
 *   - `stream` is a cudaStream_t passed as void*.  Calls only enqueue work on
 *     it and return; nothing synchronises except rs_async_status.
 *   - Errors are return codes.  Invalid arguments are detected on the host and
 *     nothing is launched.  Nothing throws, aborts or traps.  A device-side
 *     anomaly (a bounded wait that ran out) sets a status word that
 *     rs_async_status returns.
 *   - One rs_ctx per host thread.
 */
#ifndef RS_H_
#define RS_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#if defined(__GNUC__)
#define RS_API __attribute__((visibility("default")))
#else
#define RS_API
#endif

typedef enum {
    RS_OK = 0,
    RS_ERR_INVALID_ARG = 1,   /* null / misaligned pointer, size out of range              */
    RS_ERR_UNSUPPORTED = 2,   /* valid request the library has no kernel for               */
    RS_ERR_WORKSPACE = 3,     /* workspace missing or smaller than the *_workspace_bytes   */
    RS_ERR_CUDA = 4,          /* a CUDA runtime call failed; see rs_last_error             */
    RS_ERR_TIMEOUT = 5        /* a bounded device-side wait expired (rs_async_status only) */
} rs_status;

typedef enum { RS_F32 = 0, RS_BF16 = 1 } rs_dtype;

/* Distance D of Sec. 3.3 "Distance metrics". */
typedef enum { RS_DIST_L2 = 0, RS_DIST_L1 = 1, RS_DIST_COS = 2 } rs_dist;

/* Which pair of representations the block scores (Sec. 3.3 "Operation choice"). */
typedef enum {
    RS_SCORE_MLP = 0,       /* (ii)  s = D(MLP(LN(x')), x')      -- the paper's default     */
    RS_SCORE_MLP_DELTA = 1, /*       s = D(x^, x') = |MLP(LN(x'))| -- the main figure's caption
                                     read as the shift of the residual stream across the MLP */
    RS_SCORE_ATTN = 2,      /* (i)   s = D(SA(LN(x)), x)         -- shift through attention  */
    RS_SCORE_BLOCK = 3      /* (iii) s = D(x^, x)                -- shift through the block  */
} rs_score_mode;

typedef struct rs_ctx rs_ctx; /* opaque: device id, status word, last error text */

/* Create / destroy a context bound to CUDA device `device`.  rs_create
 * allocates a few bytes of device memory for the status word. */
RS_API rs_status rs_create(rs_ctx** out, int device);
RS_API void rs_destroy(rs_ctx* ctx);
/* Text of the last error on this context; never NULL; valid until the next call. */
RS_API const char* rs_last_error(const rs_ctx* ctx);
/* Synchronise `stream`, then return and clear the device status word. */
RS_API rs_status rs_async_status(rs_ctx* ctx, void* stream);
/* 1 if the tcgen05 tensor-core kernels are available for (dtype) on this context, else 0.
 * Whether a given shape runs on them is answered by the two queries below. */
RS_API int rs_uses_tensor_cores(const rs_ctx* ctx, rs_dtype dtype);
/* Which kernels a call would run, by shape (Eq. att / Eq. MLP contractions and Eq. sa): 1 = the
 * tcgen05 kernels, 0 = the fp32-FMA kernels.  The tensor-core GEMM needs RS_BF16, N % 128 == 0 and
 * K % 64 == 0; a block runs on the tensor cores only if all four of its projections qualify
 * (D % 128 == 0, D_mlp % 128 == 0).  Every other valid shape still computes the same result on
 * the fp32-FMA kernels, far slower.  With RS_REQUIRE_TC=1 in the environment at rs_create such a
 * call returns RS_ERR_UNSUPPORTED instead of taking the slow kernels. */
RS_API int rs_linear_uses_tensor_cores(const rs_ctx* ctx, rs_dtype dtype, long long M, int N, int K);

/* ---- rs_attn_fwd: Eq. sa, out = Softmax(Q K^T * scale) V per (sample, head) ----------
 * q, k, v (dev): element [b, i, h, c] lives at  b*batch_stride + i*row_stride +
 * h*head_stride + c  (strides in elements), so the three may alias one packed
 * [B, N, 3, H, 64] buffer.  Strides must be multiples of 8 elements.
 * out (dev): [B, N, H*head_dim] contiguous, same dtype.  No [N, N] buffer is
 * ever written to global memory.  scale == 0 selects 1/sqrt(head_dim).
 * Two tensor-core kernels serve bf16 (two or three 128-row query tiles per thread block); the
 * library picks the one its cost model expects to be faster for B, N and H, so the result for
 * one shape is reproducible bit for bit but the rounding order may differ between shapes.
 * RS_ATTN_KERNEL=2 or =3 in the environment at rs_create pins one of them where it applies. */
typedef struct {
    rs_dtype dtype;
    int B, N, H, head_dim;
    float scale;
    long long q_batch_stride, q_row_stride, q_head_stride;
    long long k_batch_stride, k_row_stride, k_head_stride;
    long long v_batch_stride, v_row_stride, v_head_stride;
} rs_attn_desc;

RS_API rs_status rs_attn_fwd(rs_ctx* ctx, const rs_attn_desc* desc /*host*/, const void* q, const void* k,
                      const void* v, void* out, void* stream);

/* ---- rs_linear_fwd: one projection of the block with its epilogue (Eq. sa "[Q,K,V] = xW", ----
 * Eq. att, Eq. MLP):  out[M, N] = epilogue(A[M, K] . W[N, K]^T + bias).
 *   RS_LIN_BIAS           out in `dtype`
 *   RS_LIN_BIAS_GELU      exact-erf GELU, out in `dtype`
 *   RS_LIN_BIAS_RESIDUAL  + residual[M, N] (of `dtype`), out in fp32 (the residual stream x')
 * A, W, residual, out (dev); bias (dev, fp32, may be NULL).  With RS_BF16 and N % 128 == 0,
 * K % 64 == 0 the tensor-core kernel runs, otherwise the fp32-FMA kernel. */
typedef enum { RS_LIN_BIAS = 0, RS_LIN_BIAS_GELU = 1, RS_LIN_BIAS_RESIDUAL = 2 } rs_linear_epilogue;
RS_API rs_status rs_linear_fwd(rs_ctx* ctx, rs_dtype dtype, rs_linear_epilogue epilogue, long long M, int N,
                               int K, const void* A, const void* W, const float* bias, const void* residual,
                               void* out, void* stream);

/* ---- rs_shift_score: Sec. 3.2, s[b, i] = D(after[b, i, :], before[b, i, :]) ------------
 * after, before (dev): [B, N, D] of `dtype`; scores (dev): [B, N] fp32. */
RS_API rs_status rs_shift_score(rs_ctx* ctx, rs_dtype dtype, rs_dist dist, int B, int N, int D,
                         const void* after, const void* before, float* scores, void* stream);

/* ---- rs_topk_compact: Sec. 3.1 / 3.2, drop the r lowest-score tokens of every sample ----
 * Keeps K = N - r tokens: token 0 first if has_cls, then by score descending,
 * ties to the lower index, NaN last.  keep_idx (dev, [B, K] int32) lists the
 * kept indices in ascending order; x_out[b, j, :] = x[b, keep_idx[b, j], :].
 * scores (dev): [B, N] fp32.  x (dev): [B, N, D]; x_out (dev): [B, K, D], must
 * not overlap x.  0 <= r <= N - 1, 1 <= N <= 32768.  r == 0 is a plain copy.
 * x and x_out may both be NULL to get the indices only. */
RS_API rs_status rs_topk_compact(rs_ctx* ctx, rs_dtype dtype, int B, int N, int D, int r, int has_cls,
                          const float* scores, const void* x, void* x_out, int32_t* keep_idx,
                          void* stream);

/* ---- rs_linewise_compact: Sec. 4 "CNN and SSM", line-wise variant (L-W) --------------------
 * A feature map is an H x W grid of tokens with D channels each (channels last).  The scores
 * (the representation shift of every position, e.g. from rs_shift_score on the [B, H*W, D]
 * maps before and after a stage) are averaged over every row and over every column of the
 * full grid; the drop_rows rows and drop_cols columns with the lowest averages are removed,
 * whole lines at a time, so the result is again a dense grid.  A line outranks another when
 * its average is larger, or equal with the lower index; NaN averages rank last.  Averages
 * are fp64 sums in index order divided by the line length.
 * scores (dev): [B, H, W] fp32.  x (dev): [B, H, W, D] of `dtype`; x_out (dev):
 * [B, H-drop_rows, W-drop_cols, D], must not overlap x; both may be NULL to get the indices
 * only.  keep_rows (dev): [B, H-drop_rows] int32 ascending; keep_cols (dev):
 * [B, W-drop_cols].  1 <= H, W <= 256; 0 <= drop_rows <= H-1; 0 <= drop_cols <= W-1;
 * D a multiple of 8.  Errors: RS_ERR_INVALID_ARG / RS_ERR_UNSUPPORTED before any launch. */
RS_API rs_status rs_linewise_compact(rs_ctx* ctx, rs_dtype dtype, int B, int H, int W, int D, int drop_rows,
                                     int drop_cols, const float* scores, const void* x, void* x_out,
                                     int32_t* keep_rows, int32_t* keep_cols, void* stream);

/* ---- rs_block_fwd: Eq. att + Eq. MLP + score + pruning in one call ----------------------
 * dtype: storage type of x, the weight matrices and x_out.  With RS_BF16 the
 * contractions run on the tensor cores with fp32 accumulation; the residual
 * stream x' is held in fp32 inside the block.  out_dtype: type written to
 * x_out / x_full (RS_F32 with dtype RS_BF16 gives the un-rounded result). */
typedef struct {
    rs_dtype dtype;
    rs_dtype out_dtype;
    int B, N, D, H, D_mlp;
    int r;                 /* tokens dropped after the block, 0 <= r <= N-1 */
    int has_cls;
    float ln_eps;          /* 0 => 1e-6 */
    float scale;           /* 0 => 1/sqrt(D/H) */
    rs_score_mode score_mode;
    rs_dist dist;          /* distance D of the score (Sec. 3.3 "Distance metrics") */
} rs_block_desc;

typedef struct {           /* all dev pointers */
    const void *w_qkv /*[3D,D]*/, *w_o /*[D,D]*/, *w_fc1 /*[D_mlp,D]*/, *w_fc2 /*[D,D_mlp]*/; /* dtype */
    const float *b_qkv, *b_o, *b_fc1, *b_fc2;        /* fp32; may be NULL */
    const float *ln1_g, *ln1_b, *ln2_g, *ln2_b;      /* fp32 */
    /* Optional, all three or none (NULL): the block's first LayerNorm folded into its QKV projection, as
     * rs_prepare_ln1_fold writes them.  Only rs_vit_fwd / rs_vit_fwd_taps use them. */
    const void* w_qkv_ln;    /* [3D, D] dtype: w_qkv with column k scaled by ln1_g[k] */
    const float* c_qkv_ln;   /* [3D] fp32: row sums of w_qkv_ln */
    const float* b_qkv_ln;   /* [3D] fp32: b_qkv + w_qkv . ln1_b */
} rs_block_weights;

/* ---- rs_prepare_ln1_fold: LayerNorm folded into the projection that follows it (Eq. att: the ----
 * block computes SA(LN(x)); the paper fixes the arithmetic, not where the normalisation is applied).
 * For a row x with mean mu and reciprocal standard deviation rstd over its D features,
 *   LN(x) W^T + b  =  rstd * (x W'^T - mu * c) + b',   W'[n,k] = W[n,k] g[k],  c[n] = sum_k W'[n,k],
 *   b'[n] = b[n] + sum_k W[n,k] beta[k],
 * so the projection can read the un-normalised tokens and the LayerNorm kernel (a full read and write of
 * the [T, D] activations) disappears; mu and rstd come from sums that the previous block's last
 * product leaves behind.  This call writes W' (rounded to `dtype`), c (sums of the rounded W') and b'
 * into caller buffers; put them in rs_block_weights and the layer loop uses the folded form for every
 * block but the first: the sums come from the previous block's FC2 epilogue when that block drops no
 * token, else from the kernel that moves the kept rows (which then copies them instead of normalising
 * them, into a dense buffer).  RS_BF16 only; D a multiple of 128.  Results differ from
 * the unfolded loop by rounding (W g is rounded once more, LN(x) is not rounded to bf16). */
RS_API rs_status rs_prepare_ln1_fold(rs_ctx* ctx, rs_dtype dtype, int D, const void* w_qkv, const float* b_qkv,
                                     const float* ln1_g, const float* ln1_b, void* w_out, float* c_out,
                                     float* b_out, void* stream);

/* 1 if rs_block_fwd runs this descriptor on the tcgen05 kernels, 0 if on the fp32-FMA kernels
 * (see rs_linear_uses_tensor_cores). */
RS_API int rs_block_uses_tensor_cores(const rs_ctx* ctx, const rs_block_desc* desc /*host*/);

/* Bytes of scratch rs_block_fwd needs for this descriptor (0 on a bad descriptor). */
RS_API size_t rs_block_workspace_bytes(const rs_block_desc* desc /*host*/);

/* x (dev): [B, N, D].  x_out (dev): [B, N-r, D].  scores (dev, optional):
 * [B, N] fp32.  keep_idx (dev, optional): [B, N-r] int32.  x_full (dev,
 * optional): [B, N, D] un-pruned x^ of out_dtype.  workspace (dev): at least
 * rs_block_workspace_bytes(desc) bytes, 256-byte aligned, contents undefined
 * before and after. */
RS_API rs_status rs_block_fwd(rs_ctx* ctx, const rs_block_desc* desc /*host*/,
                       const rs_block_weights* weights /*host struct of dev pointers*/,
                       const void* x, void* x_out, float* scores, int32_t* keep_idx, void* x_full,
                       void* workspace, size_t workspace_bytes, void* stream);

/* ---- rs_vit_fwd: the layer loop (Sec. 3.2: tokens are dropped after the listed blocks and ----
 * every later block runs on the reduced set).  Runs L blocks back to back on `stream`;
 * block l (0-based) drops drops[l] tokens after its MLP (0 = none), so block l+1 sees
 * N_{l+1} = N_l - drops[l] tokens.  Everything else is as in rs_block_fwd, with one
 * descriptor for the whole stack.
 * weights (host): array of L structs of dev pointers.  drops (host): L ints, each in
 * [0, N_l - 1].  x (dev): [B, N, D].  x_out (dev): [B, N_L, D] with N_L = N - sum(drops).
 * scores_last / keep_last (dev, optional): the last block's scores [B, N_{L-1}] and kept
 * indices [B, N_L].  workspace (dev): at least rs_vit_workspace_bytes() bytes, 256-byte
 * aligned; it holds one block's scratch, two token buffers the blocks alternate between, one
 * buffer for the normalised input of the next block and two row-index lists. */
typedef struct {
    rs_dtype dtype;
    int B, N, D, H, D_mlp, L;
    int has_cls;
    float ln_eps;          /* 0 => 1e-6 */
    float scale;           /* 0 => 1/sqrt(D/H) */
    rs_score_mode score_mode;
    rs_dist dist;
} rs_vit_desc;

/* Optional per-block outputs of the layer loop.  Each member is NULL or a host array of L device
 * pointers, any of which may be NULL (x_out[L-1], the result, is required).  x_out[l]: block l's
 * compacted output [B, N_{l+1}, D]; scores[l]: [B, N_l] fp32; keep_idx[l]: [B, N_{l+1}] int32. */
typedef struct {
    void* const* x_out;
    float* const* scores;
    int32_t* const* keep_idx;
} rs_vit_taps;

RS_API size_t rs_vit_workspace_bytes(const rs_vit_desc* desc /*host*/, const int* drops /*host[L]*/);
/* The layer loop with every block's outputs available.  Same computation as rs_vit_fwd.  In both,
 * the pruning kernel of a block that drops tokens also writes LN1 of the next block's input
 * (the kept row is in its registers), so a block after a pruning block launches no LN1 kernel.
 * The reduced token set of Sec. 3.1 is materialised as a dense [B, N_{l+1}, D] buffer only where a
 * caller asks for it (taps->x_out[l] non-NULL, and always for the last block): otherwise the
 * un-pruned output stays where the block wrote it and the next block reads the kept rows in place
 * through the index list (its LN1 and the residual of its projection), so the copy's
 * B * N_{l+1} * D elements are never written.  The results are the same bits either way. */
RS_API rs_status rs_vit_fwd_taps(rs_ctx* ctx, const rs_vit_desc* desc /*host*/,
                                 const rs_block_weights* weights /*host[L]*/, const int* drops /*host[L]*/,
                                 const void* x, const rs_vit_taps* taps /*host*/, void* workspace,
                                 size_t workspace_bytes, void* stream);
RS_API rs_status rs_vit_fwd(rs_ctx* ctx, const rs_vit_desc* desc /*host*/,
                            const rs_block_weights* weights /*host[L]*/, const int* drops /*host[L]*/,
                            const void* x, void* x_out, float* scores_last, int32_t* keep_last,
                            void* workspace, size_t workspace_bytes, void* stream);

/* ---- per-sample token counts (Sec. 3.1: the reduced token set, here with a count of its own per ----
 * sample, as a score threshold or a per-sample ratio gives; Sec. 4.1 "Settings" prunes by ratio).
 * Layout: padded.  Every sample owns N rows of its tensors; sample b's seq_lens[b] tokens sit at the
 * front of its rows, the rows behind them are padding.  Padding rows of an INPUT must hold finite
 * values (zeros will do): they are multiplied by zero weights, never selected.  Padding rows of the
 * token OUTPUT x_out are written as zeros, of keep_idx as -1; other outputs (attention rows, scores,
 * x_full) are unspecified but finite there.  seq_lens, drops, lens_out (dev): [B] int32.  Values are
 * read on the device and clamped there: seq_lens to [1, N], drops to [0, seq_lens[b] - 1], and the
 * kept count seq_lens[b] - drops[b] to at most the row stride of the outputs.  Tensor-core path only
 * (RS_BF16, head_dim 64; for the block D and D_mlp multiples of 128) and N <= 4608:
 * RS_ERR_UNSUPPORTED otherwise, before any launch.
 *
 * rs_attn_fwd_ragged: rs_attn_fwd where sample b attends over its first seq_lens[b] tokens (Eq. sa
 * on that many rows).
 * rs_topk_compact_ragged: rs_topk_compact where sample b drops the drops[b] lowest-score tokens of
 * its first seq_lens[b]; x_out [B, K_pad, D] and keep_idx [B, K_pad] have row stride K_pad >= every
 * kept count; lens_out (optional) receives the kept counts.
 * rs_block_fwd_ragged: rs_block_fwd on such a batch; desc->N is the padded length, desc->r fixes the
 * row stride K_pad = N - r of x_out and keep_idx (so r must not exceed any drops[b]); keep_idx is
 * required.  Workspace as for rs_block_fwd with the same descriptor. */
RS_API rs_status rs_attn_fwd_ragged(rs_ctx* ctx, const rs_attn_desc* desc /*host*/, const void* q, const void* k,
                                    const void* v, void* out, const int32_t* seq_lens, void* stream);
RS_API rs_status rs_topk_compact_ragged(rs_ctx* ctx, rs_dtype dtype, int B, int N, int D, int K_pad, int has_cls,
                                        const float* scores, const void* x, void* x_out, int32_t* keep_idx,
                                        const int32_t* seq_lens, const int32_t* drops, int32_t* lens_out,
                                        void* stream);
RS_API rs_status rs_block_fwd_ragged(rs_ctx* ctx, const rs_block_desc* desc /*host*/,
                                     const rs_block_weights* weights /*host struct of dev pointers*/, const void* x,
                                     void* x_out, float* scores, int32_t* keep_idx, void* x_full,
                                     const int32_t* seq_lens, const int32_t* drops, int32_t* lens_out,
                                     void* workspace, size_t workspace_bytes, void* stream);

/* rs_vit_fwd_ragged: the layer loop on a batch with per-sample token counts -- rs_block_fwd_ragged
 * chained L times inside the library, the same bits as chaining the calls.  pad_drops (host[L]): the
 * padded length shrinks from N_l to N_{l+1} = N_l - pad_drops[l] after block l (so pad_drops[l] must
 * not exceed any sample's own drop count there, or kept tokens are cut off at the row stride).
 * seq_lens (dev [B]): token counts entering block 0.  sample_drops (dev [L, B]): row l holds the
 * tokens each sample drops after block l (clamped on the device like drops above).  x (dev):
 * [B, N, D]; x_out (dev): [B, N_L, D]; keep_last (dev, optional): [B, N_L]; lens_out (dev, optional):
 * [B] counts after the last block.  workspace: at least rs_vit_workspace_bytes(desc, pad_drops). */
RS_API rs_status rs_vit_fwd_ragged(rs_ctx* ctx, const rs_vit_desc* desc /*host*/,
                                   const rs_block_weights* weights /*host[L]*/, const int* pad_drops /*host[L]*/,
                                   const void* x, void* x_out, int32_t* keep_last, const int32_t* seq_lens,
                                   const int32_t* sample_drops, int32_t* lens_out, void* workspace,
                                   size_t workspace_bytes, void* stream);

/* ---- rs_block_fwd_static: rs_block_fwd for callers that cannot allocate ----------------
 * (The paper has no counterpart; this is a packaging variant of rs_block_fwd.)
 * Some callers have no way to obtain device memory when they reach the block:
 * code running inside a region where cudaMalloc is forbidden or would
 * synchronise the device (a latency-critical serving loop, a plug-in that is
 * handed only its input and output buffers, a host framework whose allocator
 * the plug-in must not bypass).  This entry point needs no context and no
 * workspace: its scratch is a fixed array of RS_STATIC_SCRATCH_BYTES that is
 * part of the library image, so every GPU that loads the library holds that
 * much memory until the process exits.  It calls no cudaMalloc / cudaFree and
 * no allocating library routine.
 *
 * Arguments and results are those of rs_block_fwd (same kernels, same
 * numbers); the caller still owns x, x_out, scores, keep_idx and x_full.
 * err (host, optional): receives a message when the status is not RS_OK.
 * Limits and caveats:
 *   - rs_block_workspace_bytes(desc) must not exceed RS_STATIC_SCRATCH_BYTES,
 *     else RS_ERR_WORKSPACE is returned and nothing is launched (a ViT-S block
 *     of 2 x 197 tokens in fp32 needs about 7 MiB).
 *   - The CUDA device current at the call is used.  The first call on each
 *     device looks up the array's device address and sets a kernel attribute;
 *     make that first call before starting any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the last
 *     call left there.  Nothing in it has to start at zero (every call writes
 *     what it later reads), but two calls whose kernels overlap on the GPU --
 *     different streams, or different host threads -- race on it: serialise
 *     them on one stream. */
#define RS_STATIC_SCRATCH_BYTES (16u << 20)
RS_API size_t rs_static_scratch_bytes(void);
RS_API rs_status rs_block_fwd_static(const rs_block_desc* desc /*host*/,
                                     const rs_block_weights* weights /*host struct of dev pointers*/,
                                     const void* x, void* x_out, float* scores, int32_t* keep_idx,
                                     void* x_full, void* stream, char* err /*host*/, size_t err_len);
/* rs_async_status for the calls above (they have no context to ask): synchronises `stream`,
 * then returns and clears the status word that the kernels of rs_block_fwd_static write on the
 * current device -- RS_ERR_TIMEOUT when a bounded device-side wait ran out, RS_ERR_CUDA when a
 * kernel found its shared-memory window misaligned or a runtime call failed; in both cases the
 * outputs of the calls since the last query are not to be used.  RS_OK before the first
 * rs_block_fwd_static call on the device.  Allocates nothing (one 4-byte copy to the host). */
RS_API rs_status rs_static_async_status(void* stream, char* err /*host*/, size_t err_len);

#ifdef __cplusplus
}
#endif
#endif /* RS_H_ */
