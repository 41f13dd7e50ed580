// C ABI: argument validation, the context object and the launch sequence of
// one block (Eq. att, Eq. MLP, Sec. 3.2 score, Sec. 3.1 pruning).
#include <math.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <nvtx3/nvToolsExt.h>

#include "rs_internal.h"
#include <vector>

namespace {

rs_status fail(rs_ctx* ctx, rs_status code, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return code;
}

rs_status cuda_fail(rs_ctx* ctx, cudaError_t e, const char* what) {
    return fail(ctx, RS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool valid_dtype(int t) { return t == RS_F32 || t == RS_BF16; }

// Launch wrapper: counts the launch and, when timing is on, brackets it with events.  RS_LOG=1
// prints a line per launch on stderr, RS_NVTX=1 wraps the host side of each launch in an NVTX range
// named after the step (both read at rs_create; host-side only, nothing changes in the kernels).
#define RS_CHECK_LAUNCH(ctx, cls, st, expr, what)                                  \
    do {                                                                           \
        const bool timed__ = (ctx)->timing && (ctx)->n_events < kMaxTimed;         \
        if (timed__) cudaEventRecord((ctx)->ev[2 * (ctx)->n_events], (st));        \
        if ((ctx)->nvtx) nvtxRangePushA(what);                                     \
        cudaError_t e__ = (expr);                                                  \
        if ((ctx)->nvtx) nvtxRangePop();                                           \
        if ((ctx)->log)                                                            \
            fprintf(stderr, "rs: launch %lld class %d: %s -> %s\n", (ctx)->launches, (int)(cls), what, \
                    e__ == cudaSuccess ? "ok" : cudaGetErrorString(e__));          \
        if (e__ != cudaSuccess) return cuda_fail(ctx, e__, what);                  \
        if (timed__) {                                                             \
            cudaEventRecord((ctx)->ev[2 * (ctx)->n_events + 1], (st));             \
            (ctx)->ev_class[(ctx)->n_events++] = (unsigned char)(cls);             \
        }                                                                          \
        (ctx)->launches += 1;                                                      \
    } while (0)

// Scratch layout of one block.  Every buffer starts on a 256-byte boundary.
struct BlockWs {
    size_t u, qkv, o, x_prime, h, m, x_hat, scores, keep, flags, total;
};

bool block_layout(const rs_block_desc& d, BlockWs* ws) {
    if (!valid_dtype(d.dtype) || !valid_dtype(d.out_dtype)) return false;
    if (d.B < 1 || d.N < 1 || d.D < 8 || d.H < 1 || d.D_mlp < 8) return false;
    const size_t T = (size_t)d.B * d.N, D = d.D, Dm = d.D_mlp;
    const size_t sz = rs::dtype_size(d.dtype), osz = rs::dtype_size(d.out_dtype);
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t at = off; off += rs::align_up(bytes, 256); return at; };
    ws->u = take(T * D * sz);            // LN1 / LN2 output
    ws->qkv = take(T * 3 * D * sz);      // packed [T, 3, H, 64]
    ws->o = take(T * D * sz);            // attention output
    ws->x_prime = take(T * D * 4);       // residual stream x', fp32
    ws->h = take(T * Dm * sz);           // GELU(FC1)
    ws->m = take(T * D * 4);             // MLP(LN(x')) in fp32
    ws->x_hat = take(T * D * osz);       // un-pruned block output when the caller gives no x_full
    ws->scores = take(T * 4);            // when the caller gives no scores buffer
    ws->keep = take((size_t)d.B * (size_t)(d.N) * 4);
    ws->flags = take(T + 4 * (T / 64 + 2 * (size_t)d.B) + 16);   // slice counts and keep flags between the ranking kernel and the mover
    ws->total = off;
    return true;
}

}  // namespace

extern "C" {

rs_status rs_create(rs_ctx** out, int device) {
    if (!out) return RS_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return RS_ERR_CUDA;
    rs_ctx* ctx = (rs_ctx*)aligned_alloc(64, (sizeof(rs_ctx) + 63) / 64 * 64);
    if (!ctx) return RS_ERR_CUDA;
    memset(ctx, 0, sizeof(rs_ctx));
    ctx->device = device;
    strcpy(ctx->err, "ok");
    cudaDeviceProp prop;
    if (cudaSetDevice(device) != cudaSuccess || cudaGetDeviceProperties(&prop, device) != cudaSuccess) {
        free(ctx);
        return RS_ERR_CUDA;
    }
    if (prop.major != 10) {   // kernels are built for sm_100a only
        free(ctx);
        return RS_ERR_UNSUPPORTED;
    }
    ctx->sm_count = prop.multiProcessorCount;
    if (cudaMalloc(&ctx->d_status, 256 + kFlagScratch) != cudaSuccess || cudaMemset(ctx->d_status, 0, 256) != cudaSuccess ||
        rs::select_init() != cudaSuccess) {
        if (ctx->d_status) cudaFree(ctx->d_status);
        free(ctx);
        return RS_ERR_CUDA;
    }
    ctx->d_flags = (unsigned char*)ctx->d_status + 256;
    // RS_DISABLE_TC=1 routes bf16 through the fp32-FMA kernels (cross-check of the tcgen05 path).
    const char* no_tc = getenv("RS_DISABLE_TC");
    ctx->encode_tiled = rs::tc_get_encode_fn();
    ctx->use_tc = (ctx->encode_tiled != nullptr) && !(no_tc && no_tc[0] == '1');
    // RS_ATTN_KERNEL=2 / 3 pins the attention kernel (cross-check of the two against each other)
    const char* ak = getenv("RS_ATTN_KERNEL");
    ctx->attn_kernel = ak && (ak[0] == '2' || ak[0] == '3') ? ak[0] - '0' : 0;
    const char* lg = getenv("RS_LOG");
    ctx->log = lg && lg[0] == '1';
    const char* nv = getenv("RS_NVTX");
    ctx->nvtx = nv && nv[0] == '1';
    const char* req = getenv("RS_REQUIRE_TC");
    ctx->require_tc = req && req[0] == '1';
    *out = ctx;
    return RS_OK;
}

void rs_destroy(rs_ctx* ctx) {
    if (!ctx) return;
    cudaSetDevice(ctx->device);
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->ev) {
        for (int i = 0; i < 2 * kMaxTimed; ++i) cudaEventDestroy(ctx->ev[i]);
        free(ctx->ev);
        free(ctx->ev_class);
    }
    free(ctx);
}

rs_status rs_timing_enable(rs_ctx* ctx, int on) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (on && !ctx->ev) {
        ctx->ev = (cudaEvent_t*)calloc(2 * kMaxTimed, sizeof(cudaEvent_t));
        ctx->ev_class = (unsigned char*)calloc(kMaxTimed, 1);
        if (!ctx->ev || !ctx->ev_class) return fail(ctx, RS_ERR_CUDA, "out of host memory");
        for (int i = 0; i < 2 * kMaxTimed; ++i) {
            cudaError_t e = cudaEventCreate(&ctx->ev[i]);
            if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaEventCreate");
        }
    }
    ctx->timing = on ? 1 : 0;
    ctx->n_events = 0;
    return RS_OK;
}

rs_status rs_timing_read(rs_ctx* ctx, void* stream, double* ms, long long* launches) {
    if (!ctx || !ms || !launches) return RS_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaStreamSynchronize");
    for (int c = 0; c < RS_K_COUNT; ++c) { ms[c] = 0.0; launches[c] = 0; }
    for (int i = 0; i < ctx->n_events; ++i) {
        float t = 0.f;
        e = cudaEventElapsedTime(&t, ctx->ev[2 * i], ctx->ev[2 * i + 1]);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaEventElapsedTime");
        ms[ctx->ev_class[i]] += t;
        launches[ctx->ev_class[i]] += 1;
    }
    ctx->n_events = 0;
    return RS_OK;
}

const char* rs_last_error(const rs_ctx* ctx) { return ctx ? ctx->err : "null context"; }

rs_status rs_async_status(rs_ctx* ctx, void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    cudaError_t e = cudaStreamSynchronize((cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "cudaStreamSynchronize");
    int word = 0;
    e = cudaMemcpy(&word, ctx->d_status, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "status read");
    if (word != RS_DEV_OK) {
        cudaMemset(ctx->d_status, 0, sizeof(int));
        if (word == RS_DEV_SMEM_ALIGN)
            return fail(ctx, RS_ERR_CUDA, "device status word = %d (a kernel's shared memory window was not 1024-byte aligned)", word);
        return fail(ctx, RS_ERR_TIMEOUT, "device status word = %d (a bounded wait expired)", word);
    }
    return RS_OK;
}

int rs_uses_tensor_cores(const rs_ctx* ctx, rs_dtype dtype) {
    return ctx && ctx->use_tc && dtype == RS_BF16;
}

long long rs_launch_count(const rs_ctx* ctx) { return ctx ? ctx->launches : 0; }

int rs_attn_kernel_choice(int sm_count, int B, int H, int N) {
    if (sm_count < 1 || B < 1 || H < 1 || N < 1) return 0;
    if (N <= 128) return 2;
    return rs::attn_plan((long long)B * H, N, sm_count).three ? 3 : 2;
}

rs_status rs_tmap_cache_stats(const rs_ctx* ctx, long long* hits, long long* misses) {
    if (!ctx || !hits || !misses) return RS_ERR_INVALID_ARG;
    *hits = ctx->tmap_hits;
    *misses = ctx->tmap_misses;
    return RS_OK;
}

int rs_linear_uses_tensor_cores(const rs_ctx* ctx, rs_dtype dtype, long long M, int N, int K) {
    return ctx && ctx->use_tc && dtype == RS_BF16 && rs::gemm_tc_supported(M, N, K);
}

int rs_block_uses_tensor_cores(const rs_ctx* ctx, const rs_block_desc* d) {
    if (!ctx || !d || !ctx->use_tc || d->dtype != RS_BF16 || d->B < 1 || d->N < 1) return 0;
    const long long T = (long long)d->B * d->N;
    return rs::gemm_tc_supported(T, 3 * d->D, d->D) && rs::gemm_tc_supported(T, d->D, d->D) &&
           rs::gemm_tc_supported(T, d->D_mlp, d->D) && rs::gemm_tc_supported(T, d->D, d->D_mlp);
}

rs_status rs_attn_fwd(rs_ctx* ctx, const rs_attn_desc* d, const void* q, const void* k, const void* v,
                      void* out, void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!d || !q || !k || !v || !out) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd: null argument");
    if (!valid_dtype(d->dtype)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd: bad dtype");
    if (d->B < 1 || d->N < 1 || d->H < 1) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd: B, N, H must be >= 1");
    if (d->head_dim != 64) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_attn_fwd: head_dim must be 64");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd: pointers must be 16-byte aligned");
    const long long st[9] = {d->q_batch_stride, d->q_row_stride, d->q_head_stride, d->k_batch_stride,
                             d->k_row_stride,   d->k_head_stride, d->v_batch_stride, d->v_row_stride,
                             d->v_head_stride};
    for (int i = 0; i < 9; ++i)
        if (st[i] < 0 || (st[i] % 8) != 0) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd: strides must be non-negative multiples of 8");
    if (!(d->scale >= 0.f)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd: scale must be >= 0");
    if (ctx->use_tc && rs::attn_tc_supported(*d))
        RS_CHECK_LAUNCH(ctx, RS_K_ATTN, (cudaStream_t)stream, rs::launch_attn_tc(ctx, *d, q, k, v, out, nullptr, (cudaStream_t)stream), "tensor-core attention launch");
    else
        RS_CHECK_LAUNCH(ctx, RS_K_ATTN, (cudaStream_t)stream, rs::launch_attn_simt(*d, q, k, v, out, (cudaStream_t)stream), "attention launch");
    return RS_OK;
}

rs_status rs_linear_fwd(rs_ctx* ctx, rs_dtype dtype, rs_linear_epilogue epi, long long M, int N, int K,
                        const void* A, const void* W, const float* bias, const void* residual, void* out,
                        void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!valid_dtype(dtype) || epi < RS_LIN_BIAS || epi > RS_LIN_BIAS_RESIDUAL)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_linear_fwd: bad dtype or epilogue");
    if (M < 0 || N < 8 || K < 8 || (N % 8) || (K % 8) || M >= (1ll << 31))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_linear_fwd: need M >= 0 and N, K positive multiples of 8");
    if (M == 0) return RS_OK;
    if (!A || !W || !out || (epi == RS_LIN_BIAS_RESIDUAL && !residual))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_linear_fwd: null pointer");
    if (!aligned16(A) || !aligned16(W) || !aligned16(out) || !aligned16(bias) || !aligned16(residual))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_linear_fwd: pointers must be 16-byte aligned");
    cudaStream_t st = (cudaStream_t)stream;
    const rs_dtype out_dtype = epi == RS_LIN_BIAS_RESIDUAL ? RS_F32 : dtype;
    if (ctx->require_tc && dtype == RS_BF16 && !rs_linear_uses_tensor_cores(ctx, dtype, M, N, K))
        return fail(ctx, RS_ERR_UNSUPPORTED, "rs_linear_fwd: shape outside the tensor-core kernel (N %% 128, K %% 64) and RS_REQUIRE_TC is set");
    if (ctx->use_tc && dtype == RS_BF16 && rs::gemm_tc_supported(M, N, K)) {
        const int e = epi == RS_LIN_BIAS ? rs::RS_EPI_BIAS : epi == RS_LIN_BIAS_GELU ? rs::RS_EPI_BIAS_GELU : rs::RS_EPI_RESID;
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_tc(ctx, e, A, W, bias, residual, nullptr, nullptr, out, out_dtype, nullptr, 0, 0, M, N, K, st), "tensor-core GEMM");
    } else {
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_simt(dtype, A, W, bias, epi == RS_LIN_BIAS_GELU, epi == RS_LIN_BIAS_RESIDUAL ? residual : nullptr, dtype, out, out_dtype, M, N, K, st), "GEMM");
    }
    return RS_OK;
}

rs_status rs_shift_score(rs_ctx* ctx, rs_dtype dtype, rs_dist dist, int B, int N, int D, const void* after,
                         const void* before, float* scores, void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!valid_dtype(dtype) || dist < RS_DIST_L2 || dist > RS_DIST_COS)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_shift_score: bad dtype or distance");
    if (B < 0 || N < 0 || D < 8 || (D % 8) != 0) return fail(ctx, RS_ERR_INVALID_ARG, "rs_shift_score: need B, N >= 0 and D a positive multiple of 8");
    if ((long long)B * N == 0) return RS_OK;
    if (!after || !before || !scores) return fail(ctx, RS_ERR_INVALID_ARG, "rs_shift_score: null pointer");
    if (!aligned16(after) || !aligned16(before) || (reinterpret_cast<uintptr_t>(scores) & 3u))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_shift_score: misaligned pointer");
    RS_CHECK_LAUNCH(ctx, RS_K_SCORE, (cudaStream_t)stream, rs::launch_shift_score(dtype, dist, (long long)B * N, D, after, before, scores, (cudaStream_t)stream),
                    "shift score launch");
    return RS_OK;
}

rs_status rs_topk_compact(rs_ctx* ctx, rs_dtype dtype, int B, int N, int D, int r, int has_cls,
                          const float* scores, const void* x, void* x_out, int32_t* keep_idx, void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact: bad dtype");
    if (B < 0 || N < 1) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact: need B >= 0, N >= 1");
    if (N > 32768) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_topk_compact: N > 32768");
    if (r < 0 || r > N - 1) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact: need 0 <= r <= N-1");
    if (B == 0) return RS_OK;
    if (!scores || !keep_idx) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact: null scores or keep_idx");
    if ((x == nullptr) != (x_out == nullptr)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact: x and x_out must both be given or both be NULL");
    const int K = N - r;
    cudaStream_t st = (cudaStream_t)stream;
    if (x) {
        if (D < 8 || (D % 8) != 0) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact: D must be a positive multiple of 8");
        if (!aligned16(x) || !aligned16(x_out)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact: misaligned pointer");
        const size_t sz = rs::dtype_size(dtype);
        const char* xa = (const char*)x;
        const char* xo = (const char*)x_out;
        const size_t xbytes = (size_t)B * N * D * sz, obytes = (size_t)B * K * D * sz;
        if (xa < xo + obytes && xo < xa + xbytes) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact: x_out overlaps x");
    }
    int nl = 1;
    if (x && rs::prune_fusable(N, K, kFlagScratch)) {
        RS_CHECK_LAUNCH(ctx, RS_K_GATHER, st, rs::launch_prune(scores, 0, nullptr, B, N, K, has_cls ? 1 : 0, keep_idx, nullptr, dtype, x, D, x_out, nullptr, ctx->d_flags, kFlagScratch, ctx->sm_count, st, &nl, nullptr, nullptr, nullptr), "select+gather launch");
        ctx->launches += nl - 1;
        return RS_OK;
    }
    RS_CHECK_LAUNCH(ctx, RS_K_SELECT, st, rs::launch_select(scores, 0, nullptr, B, N, K, has_cls ? 1 : 0, keep_idx, nullptr, ctx->d_flags, kFlagScratch, ctx->sm_count, st, &nl), "select launch");
    ctx->launches += nl - 1;
    if (x) RS_CHECK_LAUNCH(ctx, RS_K_GATHER, st, rs::launch_gather(dtype, x, keep_idx, B, N, K, D, x_out, nullptr, st), "gather launch");
    return RS_OK;
}

size_t rs_block_workspace_bytes(const rs_block_desc* d) {
    BlockWs ws;
    if (!d || !block_layout(*d, &ws)) return 0;
    return ws.total;
}

rs_status rs_linewise_compact(rs_ctx* ctx, rs_dtype dtype, int B, int H, int W, int D, int drop_rows, int drop_cols,
                              const float* scores, const void* x, void* x_out, int32_t* keep_rows,
                              int32_t* keep_cols, void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_linewise_compact: bad dtype");
    if (B < 0 || H < 1 || W < 1) return fail(ctx, RS_ERR_INVALID_ARG, "rs_linewise_compact: need B >= 0, H >= 1, W >= 1");
    if (H > rs::linewise_max_lines() || W > rs::linewise_max_lines())
        return fail(ctx, RS_ERR_UNSUPPORTED, "rs_linewise_compact: H and W up to %d", rs::linewise_max_lines());
    if (drop_rows < 0 || drop_rows > H - 1 || drop_cols < 0 || drop_cols > W - 1)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_linewise_compact: need 0 <= drop_rows <= H-1 and 0 <= drop_cols <= W-1");
    if (B == 0) return RS_OK;
    if (!scores || !keep_rows || !keep_cols) return fail(ctx, RS_ERR_INVALID_ARG, "rs_linewise_compact: null scores or index list");
    if ((x == nullptr) != (x_out == nullptr))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_linewise_compact: x and x_out must both be given or both be NULL");
    const int Hk = H - drop_rows, Wk = W - drop_cols;
    if (x) {
        if (D < 8 || (D % 8) != 0) return fail(ctx, RS_ERR_INVALID_ARG, "rs_linewise_compact: D must be a positive multiple of 8");
        if (!aligned16(x) || !aligned16(x_out)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_linewise_compact: misaligned pointer");
        const size_t sz = rs::dtype_size(dtype);
        const char* xa = (const char*)x;
        const char* xo = (const char*)x_out;
        const size_t xbytes = (size_t)B * H * W * D * sz, obytes = (size_t)B * Hk * Wk * D * sz;
        if (xa < xo + obytes && xo < xa + xbytes) return fail(ctx, RS_ERR_INVALID_ARG, "rs_linewise_compact: x_out overlaps x");
    }
    cudaStream_t st = (cudaStream_t)stream;
    RS_CHECK_LAUNCH(ctx, RS_K_GATHER, st, rs::launch_linewise(scores, B, H, W, Hk, Wk, keep_rows, keep_cols, dtype, x, D, x_out, ctx->sm_count, st),
                    "line-wise select+gather launch");
    return RS_OK;
}

// What the layer loop adds to a block call.
//   in_map:  the block input is read in place from the previous block's un-pruned output: row t of
//            the input is row in_map[t] of `x` ([B, N_prev, D]); null: `x` is the dense [B, N, D] input.
//   x_ln:    LN1 of the input, already computed by the previous block's pruning kernel; null: not.
//   next_ln: asks that kernel for LN of this block's kept rows with the next block's LN1 parameters
//            (it cannot when nothing is dropped or a row does not fit one warp's registers; *ln_done tells).
//   out_map: where to leave this block's row map (b * N + kept token) for the next block; with it and
//            dense_out == false the dense copy x_out is not written at all: the next block reads x^
//            through the map (Sec. 3.1: the reduced token set as an index list).
//   seq_lens, drops, lens_out: per-sample token counts (rs_block_fwd_ragged); null otherwise.
struct LoopHooks {
    const int32_t* in_map;
    const void* x_ln;
    const rs::LnFuse* next_ln;
    int32_t* out_map;
    bool dense_out;
    bool* ln_done;
    const int32_t* seq_lens;
    const int32_t* drops;
    int32_t* lens_out;
    // LN1 folded into QKV (the layer loop, blocks whose predecessor drops nothing and whose weights carry
    // the folded form): stats_in / parts_in = the row sums the previous block's FC2 left of this block's
    // input; stats_out / parts_out = where this block's FC2 leaves them for the next block.
    const float* stats_in;
    int parts_in;
    float* stats_out;
    int* parts_out;
};

static rs_status block_fwd_impl(rs_ctx* ctx, const rs_block_desc* d, const rs_block_weights* w, const void* x,
                                void* x_out, float* scores, int32_t* keep_idx, void* x_full, void* workspace,
                                size_t workspace_bytes, void* stream, const LoopHooks* hk) {
    if (hk && hk->ln_done) *hk->ln_done = false;
    if (!ctx) return RS_ERR_INVALID_ARG;
    const bool dense_out = !hk || hk->dense_out;
    if (!d || !w || !x || (dense_out && !x_out)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: null argument");
    BlockWs ws;
    if (!block_layout(*d, &ws)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: bad descriptor");
    if (d->H * 64 != d->D) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_block_fwd: D must equal 64 * H");
    if ((d->D % 8) || (d->D_mlp % 8)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: D and D_mlp must be multiples of 8");
    if (d->D > 2048 && d->dtype == RS_BF16) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_block_fwd: D > 2048");
    if (d->D > 1024 && d->dtype == RS_F32) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_block_fwd: D > 1024 in fp32");
    if (d->N > 32768) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_block_fwd: N > 32768");
    if (d->r < 0 || d->r > d->N - 1) return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: need 0 <= r <= N-1");
    if (!(d->scale >= 0.f)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: scale must be >= 0");
    if (d->dist < RS_DIST_L2 || d->dist > RS_DIST_COS) return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: bad dist");
    if (d->score_mode < RS_SCORE_MLP || d->score_mode > RS_SCORE_BLOCK)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: bad score_mode");
    if (d->dtype == RS_F32 && d->out_dtype != RS_F32)
        return fail(ctx, RS_ERR_UNSUPPORTED, "rs_block_fwd: fp32 storage writes fp32 outputs");
    if (!w->w_qkv || !w->w_o || !w->w_fc1 || !w->w_fc2 || !w->ln1_g || !w->ln1_b || !w->ln2_g || !w->ln2_b)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: null weight");
    const void* ptrs[] = {x, x_out, x_full, workspace, w->w_qkv, w->w_o, w->w_fc1, w->w_fc2, w->b_qkv, w->b_o,
                          w->b_fc1, w->b_fc2, w->ln1_g, w->ln1_b, w->ln2_g, w->ln2_b};
    for (const void* p : ptrs)
        if (p && !aligned16(p)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: pointers must be 16-byte aligned");
    if (!workspace || workspace_bytes < ws.total)
        return fail(ctx, RS_ERR_WORKSPACE, "rs_block_fwd: workspace of %zu bytes needed, %zu given", ws.total, workspace_bytes);
    if (reinterpret_cast<uintptr_t>(workspace) & 255u)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd: workspace must be 256-byte aligned");

    cudaStream_t st = (cudaStream_t)stream;
    char* base = (char*)workspace;
    const long long T = (long long)d->B * d->N;
    const int D = d->D, Dm = d->D_mlp, K = d->N - d->r;
    const float eps = d->ln_eps > 0.f ? d->ln_eps : 1e-6f;
    void* u = base + ws.u;
    void* qkv = base + ws.qkv;
    void* o = base + ws.o;
    float* x_prime = (float*)(base + ws.x_prime);
    void* h = base + ws.h;
    float* m = (float*)(base + ws.m);
    float* s = scores ? scores : (float*)(base + ws.scores);
    int32_t* keep = keep_idx ? keep_idx : (int32_t*)(base + ws.keep);
    // The un-pruned output goes to x_full if given, straight to x_out when nothing is
    // dropped, else to scratch.
    const bool ragged = hk && hk->seq_lens;
    void* x_hat = x_full ? x_full : ((d->r == 0 && !ragged) ? x_out : (void*)(base + ws.x_hat));

    const bool tc = rs_block_uses_tensor_cores(ctx, d) != 0;
    if (ctx->require_tc && d->dtype == RS_BF16 && !tc)
        return fail(ctx, RS_ERR_UNSUPPORTED, "rs_block_fwd: shape outside the tensor-core kernels (D, D_mlp multiples of 128) and RS_REQUIRE_TC is set");
    const int32_t* in_map = hk ? hk->in_map : nullptr;
    if (in_map && !tc) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_block_fwd: a row-mapped input needs the tensor-core kernels");
    if (ragged && (!tc || d->N > 4608)) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_block_fwd_ragged: needs the tensor-core kernels (bf16, D and D_mlp multiples of 128) and N <= 4608");
    const size_t sz = rs::dtype_size(d->dtype);
    rs_attn_desc ad;
    ad.dtype = d->dtype; ad.B = d->B; ad.N = d->N; ad.H = d->H; ad.head_dim = 64; ad.scale = d->scale;
    ad.q_batch_stride = ad.k_batch_stride = ad.v_batch_stride = (long long)d->N * 3 * D;
    ad.q_row_stride = ad.k_row_stride = ad.v_row_stride = 3 * D;
    ad.q_head_stride = ad.k_head_stride = ad.v_head_stride = 64;
    const void* kp = (char*)qkv + (size_t)D * sz;
    const void* vp = (char*)qkv + 2 * (size_t)D * sz;
    int nparts = 0;

    // x' = SA(LN(x)) + x                                                  (Eq. att)
    const void* x_ln = hk ? hk->x_ln : nullptr;
    const bool fold_ln1 = tc && hk && hk->stats_in && !x_ln && !in_map && w->w_qkv_ln && w->c_qkv_ln && w->b_qkv_ln;
    if (!x_ln && !fold_ln1) {
        RS_CHECK_LAUNCH(ctx, RS_K_LAYERNORM, st, rs::launch_layernorm(d->dtype, d->dtype, x, w->ln1_g, w->ln1_b, eps, T, D, u, in_map, st), "LN1");
        x_ln = u;
    }
    if (tc) {
        if (fold_ln1) {
            // LN1 applied in the epilogue: the product reads the block input itself
            const rs::GemmLn ln = {nullptr, nullptr, hk->stats_in, hk->parts_in, w->c_qkv_ln, eps};
            RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_tc(ctx, rs::RS_EPI_BIAS, x, w->w_qkv_ln, w->b_qkv_ln, nullptr, nullptr, nullptr, qkv, RS_BF16, nullptr, 0, 0, T, 3 * D, D, st, &ln), "LN1+QKV");
        } else {
            RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_tc(ctx, rs::RS_EPI_BIAS, x_ln, w->w_qkv, w->b_qkv, nullptr, nullptr, nullptr, qkv, RS_BF16, nullptr, 0, 0, T, 3 * D, D, st), "QKV");
        }
        RS_CHECK_LAUNCH(ctx, RS_K_ATTN, st, rs::launch_attn_tc(ctx, ad, qkv, kp, vp, o, hk ? hk->seq_lens : nullptr, st), "attention");
        // shift through attention (operation choice (i)): partial sums of (SA(LN(x)) - x)^2 from this epilogue
        nparts = rs::gemm_tc_score_parts(ctx, T, D);
        float* attn_parts = d->score_mode == RS_SCORE_ATTN ? m : nullptr;
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_tc(ctx, rs::RS_EPI_RESID, o, w->w_o, w->b_o, x, nullptr, in_map, x_prime, RS_F32, attn_parts, 0, (int)d->dist, T, D, D, st), "proj");
    } else {
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_simt(d->dtype, x_ln, w->w_qkv, w->b_qkv, 0, nullptr, RS_F32, qkv, d->dtype, T, 3 * D, D, st), "QKV");
        RS_CHECK_LAUNCH(ctx, RS_K_ATTN, st, rs::launch_attn_simt(ad, qkv, kp, vp, o, st), "attention");
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_simt(d->dtype, o, w->w_o, w->b_o, 0, x, d->dtype, x_prime, RS_F32, T, D, D, st), "proj");
    }
    // x^ = MLP(LN(x')) + x',  s = |MLP(LN(x')) - x'|                      (Eq. MLP, Sec. 3.2)
    RS_CHECK_LAUNCH(ctx, RS_K_LAYERNORM, st, rs::launch_layernorm(RS_F32, d->dtype, x_prime, w->ln2_g, w->ln2_b, eps, T, D, u, nullptr, st), "LN2");
    if (tc) {
        // The FC2 epilogue adds the residual and leaves per-tile partial sums of squares of the
        // shift in `m`; the selection kernel adds them up in a fixed order.
        // (when the score came from the projection, this epilogue's partial sums go to a second array)
        float* fc2_parts = d->score_mode == RS_SCORE_ATTN ? m + (size_t)T * nparts * 3 : m;
        const int kind = d->score_mode == RS_SCORE_MLP_DELTA ? 1 : d->score_mode == RS_SCORE_BLOCK ? 2 : 0;
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_tc(ctx, rs::RS_EPI_BIAS_GELU, u, w->w_fc1, w->b_fc1, nullptr, nullptr, nullptr, h, RS_BF16, nullptr, 0, 0, T, Dm, D, st), "FC1");
        // row sums for a LayerNorm folded into the next block's QKV: from this epilogue when the block's output is
        // the next block's input as it stands, else from the kernel that moves the kept rows (below)
        const bool fc2_stats = hk && hk->stats_out && x_hat == x_out;
        const rs::GemmLn lnout = {fc2_stats ? hk->stats_out : nullptr, fc2_stats ? hk->parts_out : nullptr, nullptr, 0, nullptr, 0.f};
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_tc(ctx, rs::RS_EPI_SCORE, h, w->w_fc2, w->b_fc2, x_prime, x, in_map, x_hat, d->out_dtype, fc2_parts, kind, (int)d->dist, T, D, Dm, st, fc2_stats ? &lnout : nullptr), "FC2+residual+score");
    } else {
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_simt(d->dtype, u, w->w_fc1, w->b_fc1, 1, nullptr, RS_F32, h, d->dtype, T, Dm, D, st), "FC1");
        RS_CHECK_LAUNCH(ctx, RS_K_GEMM, st, rs::launch_gemm_simt(d->dtype, h, w->w_fc2, w->b_fc2, 0, nullptr, RS_F32, m, RS_F32, T, D, Dm, st), "FC2");
        RS_CHECK_LAUNCH(ctx, RS_K_SCORE, st, rs::launch_residual_score(m, x_prime, x, d->dtype, T, D, d->score_mode, d->dist, d->out_dtype, x_hat, s, st), "residual+score");
    }
    // reduced token set                                                   (Sec. 3.1)
    const float* sel_in = nparts > 0 ? m : s;
    const int sel_enc = nparts > 0 ? (nparts | ((int)d->dist << 16)) : 0;
    float* sel_out = nparts > 0 ? s : nullptr;
    const bool moves = x_hat != x_out;      // something is dropped: the kept rows are moved (or normalised) here
    const rs::LnFuse* ln = (hk && hk->next_ln && moves && rs::ln_fusable(d->out_dtype, D)) ? hk->next_ln : nullptr;
    if (ln && hk->ln_done) *hk->ln_done = true;
    // the kept rows' sums for a LayerNorm folded into the next block's QKV (one pair per row)
    rs::LnFuse sums = {nullptr, nullptr, 0.f, nullptr, nullptr};
    if (!ln && tc && moves && dense_out && hk && hk->stats_out && !ragged && d->out_dtype == RS_BF16) {
        sums.stats = hk->stats_out;
        ln = &sums;
        if (hk->parts_out) *hk->parts_out = 1;
    }
    int32_t* out_map = (hk && moves) ? hk->out_map : nullptr;
    void* dense = dense_out ? x_out : nullptr;
    const int cls = d->has_cls ? 1 : 0;
    uint8_t* flags = (uint8_t*)(base + ws.flags);
    if (ragged) {
        // per-sample counts: sample b keeps lens[b] - drops[b] of its first lens[b] tokens; K is the row stride
        int nlr = 0;
        const size_t fb = (size_t)T + 4 * ((size_t)T / 64 + 2 * (size_t)d->B) + 16;
        RS_CHECK_LAUNCH(ctx, RS_K_GATHER, st, rs::launch_prune(sel_in, sel_enc, sel_out, d->B, d->N, K, cls, keep, nullptr, d->out_dtype, x_hat, D, x_out, nullptr, flags, fb, ctx->sm_count, st, &nlr, hk->seq_lens, hk->drops, hk->lens_out), "select+gather (per-sample counts)");
        ctx->launches += nlr - 1;
        return RS_OK;
    }
    const size_t flags_bytes = (size_t)T + 4 * ((size_t)T / 64 + 2 * (size_t)d->B) + 16;
    int nl = 1;
    if (moves && rs::prune_fusable(d->N, K, flags_bytes) && (dense || ln)) {
        RS_CHECK_LAUNCH(ctx, RS_K_GATHER, st, rs::launch_prune(sel_in, sel_enc, sel_out, d->B, d->N, K, cls, keep, out_map, d->out_dtype, x_hat, D, dense, ln, flags, flags_bytes, ctx->sm_count, st, &nl, nullptr, nullptr, nullptr), "select+gather");
        ctx->launches += nl - 1;
        return RS_OK;
    }
    // nothing dropped and neither the scores nor the (identity) index list asked for: nothing left to do
    if (!moves && hk && !scores && !keep_idx) return RS_OK;
    RS_CHECK_LAUNCH(ctx, RS_K_SELECT, st, rs::launch_select(sel_in, sel_enc, sel_out, d->B, d->N, K, cls, keep, out_map, flags, flags_bytes, ctx->sm_count, st, &nl), "select");
    ctx->launches += nl - 1;
    if (moves && (dense || ln))
        RS_CHECK_LAUNCH(ctx, RS_K_GATHER, st, rs::launch_gather(d->out_dtype, x_hat, keep, d->B, d->N, K, D, dense, ln, st), "gather");
    return RS_OK;
}

rs_status rs_block_fwd(rs_ctx* ctx, const rs_block_desc* d, const rs_block_weights* w, const void* x,
                       void* x_out, float* scores, int32_t* keep_idx, void* x_full, void* workspace,
                       size_t workspace_bytes, void* stream) {
    return block_fwd_impl(ctx, d, w, x, x_out, scores, keep_idx, x_full, workspace, workspace_bytes, stream, nullptr);
}

rs_status rs_block_fwd_ragged(rs_ctx* ctx, const rs_block_desc* d, const rs_block_weights* w, const void* x,
                              void* x_out, float* scores, int32_t* keep_idx, void* x_full, const int32_t* seq_lens,
                              const int32_t* drops, int32_t* lens_out, void* workspace, size_t workspace_bytes,
                              void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!seq_lens || !drops || !keep_idx) return fail(ctx, RS_ERR_INVALID_ARG, "rs_block_fwd_ragged: seq_lens, drops and keep_idx are required");
    const LoopHooks hk = {nullptr, nullptr, nullptr, nullptr, true, nullptr, seq_lens, drops, lens_out, nullptr, 0, nullptr, nullptr};
    return block_fwd_impl(ctx, d, w, x, x_out, scores, keep_idx, x_full, workspace, workspace_bytes, stream, &hk);
}

rs_status rs_attn_fwd_ragged(rs_ctx* ctx, const rs_attn_desc* d, const void* q, const void* k, const void* v,
                             void* out, const int32_t* seq_lens, void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!seq_lens) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd_ragged: null seq_lens");
    if (!d || !q || !k || !v || !out) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd_ragged: null argument");
    if (!valid_dtype(d->dtype) || d->B < 1 || d->N < 1 || d->H < 1) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd_ragged: bad descriptor");
    if (!aligned16(q) || !aligned16(k) || !aligned16(v) || !aligned16(out) || (reinterpret_cast<uintptr_t>(seq_lens) & 3u))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd_ragged: misaligned pointer");
    if (!(d->scale >= 0.f)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_attn_fwd_ragged: scale must be >= 0");
    if (!ctx->use_tc || !rs::attn_tc_supported(*d))
        return fail(ctx, RS_ERR_UNSUPPORTED, "rs_attn_fwd_ragged: needs the tensor-core kernel (bf16, head_dim 64, strides multiples of 8)");
    RS_CHECK_LAUNCH(ctx, RS_K_ATTN, (cudaStream_t)stream, rs::launch_attn_tc(ctx, *d, q, k, v, out, seq_lens, (cudaStream_t)stream), "tensor-core attention launch");
    return RS_OK;
}

rs_status rs_topk_compact_ragged(rs_ctx* ctx, rs_dtype dtype, int B, int N, int D, int K_pad, int has_cls,
                                 const float* scores, const void* x, void* x_out, int32_t* keep_idx,
                                 const int32_t* seq_lens, const int32_t* drops, int32_t* lens_out, void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!valid_dtype(dtype)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact_ragged: bad dtype");
    if (B < 0 || N < 1 || K_pad < 1 || K_pad > N) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact_ragged: need B >= 0, 1 <= K_pad <= N");
    if (N > 4608) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_topk_compact_ragged: N > 4608");
    if (B == 0) return RS_OK;
    if (!scores || !keep_idx || !seq_lens || !drops) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact_ragged: null scores, keep_idx, seq_lens or drops");
    if ((x == nullptr) != (x_out == nullptr)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact_ragged: x and x_out must both be given or both be NULL");
    if (x) {
        if (D < 8 || (D % 8) != 0) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact_ragged: D must be a positive multiple of 8");
        if (!aligned16(x) || !aligned16(x_out)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact_ragged: misaligned pointer");
        const size_t sz = rs::dtype_size(dtype);
        const char* xa = (const char*)x;
        const char* xo = (const char*)x_out;
        const size_t xbytes = (size_t)B * N * D * sz, obytes = (size_t)B * K_pad * D * sz;
        if (xa < xo + obytes && xo < xa + xbytes) return fail(ctx, RS_ERR_INVALID_ARG, "rs_topk_compact_ragged: x_out overlaps x");
    }
    int nl = 1;
    cudaStream_t st = (cudaStream_t)stream;
    RS_CHECK_LAUNCH(ctx, RS_K_GATHER, st, rs::launch_prune(scores, 0, nullptr, B, N, K_pad, has_cls ? 1 : 0, keep_idx, nullptr, dtype, x, D, x_out, nullptr, ctx->d_flags, kFlagScratch, ctx->sm_count, st, &nl, seq_lens, drops, lens_out), "select+gather launch (per-sample counts)");
    ctx->launches += nl - 1;
    return RS_OK;
}

}  // extern "C"

namespace {

// Plan of the layer loop: per-block descriptors, the largest block scratch and the size of one
// of the two token buffers the blocks alternate between.  False on a bad descriptor / schedule.
struct VitPlan { size_t block_ws, act_bytes, map_bytes, stats_bytes, total; int n_final; };

bool vit_plan(const rs_vit_desc& d, const int* drops, VitPlan* p) {
    if (!drops || d.L < 1 || d.B < 1 || d.N < 1) return false;
    size_t block_ws = 0;
    int n = d.N;
    for (int l = 0; l < d.L; ++l) {
        if (drops[l] < 0 || drops[l] > n - 1) return false;
        rs_block_desc bd = {d.dtype, d.dtype, d.B, n, d.D, d.H, d.D_mlp, drops[l], d.has_cls, d.ln_eps, d.scale, d.score_mode, d.dist};
        const size_t w = rs_block_workspace_bytes(&bd);
        if (w == 0) return false;
        if (w > block_ws) block_ws = w;
        n -= drops[l];
    }
    p->block_ws = rs::align_up(block_ws, 256);
    p->act_bytes = rs::align_up((size_t)d.B * d.N * d.D * rs::dtype_size(d.dtype), 256);
    p->map_bytes = rs::align_up((size_t)d.B * d.N * sizeof(int32_t), 256);
    // row sums for a LayerNorm folded into the next block's QKV: up to 2 * D / 128 pairs of floats per row
    p->stats_bytes = rs::align_up((size_t)d.B * d.N * (2 * (size_t)d.D / 128 + 2) * 8, 256);
    // block scratch, two token buffers, one LN buffer, two row maps, two row-sum buffers
    p->total = p->block_ws + 3 * p->act_bytes + 2 * p->map_bytes + 2 * p->stats_bytes;
    p->n_final = n;
    return true;
}

}  // namespace

extern "C" {

size_t rs_vit_workspace_bytes(const rs_vit_desc* d, const int* drops) {
    VitPlan p;
    if (!d || !valid_dtype(d->dtype) || !vit_plan(*d, drops, &p)) return 0;
    return p.total;
}

rs_status rs_vit_fwd_taps(rs_ctx* ctx, const rs_vit_desc* d, const rs_block_weights* weights, const int* drops,
                          const void* x, const rs_vit_taps* taps, void* workspace, size_t workspace_bytes,
                          void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!d || !weights || !drops || !x || !taps || d->L < 1 || !taps->x_out || !taps->x_out[d->L - 1])
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_vit_fwd: null argument (the last block's x_out is required)");
    VitPlan p;
    if (!valid_dtype(d->dtype) || !vit_plan(*d, drops, &p))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_vit_fwd: bad descriptor or schedule (need 0 <= drops[l] <= N_l - 1)");
    if (!workspace || workspace_bytes < p.total)
        return fail(ctx, RS_ERR_WORKSPACE, "rs_vit_fwd: workspace of %zu bytes needed, %zu given", p.total, workspace_bytes);
    if (reinterpret_cast<uintptr_t>(workspace) & 255u)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_vit_fwd: workspace must be 256-byte aligned");
    char* base = (char*)workspace;
    void* act[2] = {base + p.block_ws, base + p.block_ws + p.act_bytes};
    void* ln_buf = base + p.block_ws + 2 * p.act_bytes;   // LN1 of the next block's input, from the pruning kernel
    int32_t* maps[2] = {(int32_t*)(base + p.block_ws + 3 * p.act_bytes), (int32_t*)(base + p.block_ws + 3 * p.act_bytes + p.map_bytes)};
    float* stats[2] = {(float*)(base + p.block_ws + 3 * p.act_bytes + 2 * p.map_bytes),
                       (float*)(base + p.block_ws + 3 * p.act_bytes + 2 * p.map_bytes + p.stats_bytes)};
    const float* cur_stats = nullptr;    // row sums of the block input, when the previous block's FC2 left them
    int cur_parts = 0;
    const float eps = d->ln_eps > 0.f ? d->ln_eps : 1e-6f;
    const void* cur = x;                 // the block input: dense [B, n, D], or, with cur_map, the previous
    const int32_t* cur_map = nullptr;    // block's un-pruned x^ read through the row map
    const void* cur_ln = nullptr;
    int n = d->N;
    for (int l = 0; l < d->L; ++l) {
        const bool last = l == d->L - 1;
        rs_block_desc bd = {d->dtype, d->dtype, d->B, n, d->D, d->H, d->D_mlp, drops[l], d->has_cls, d->ln_eps, d->scale,
                            d->score_mode, d->dist};
        // A block that drops tokens and whose compacted output nobody asked for writes no dense copy:
        // its un-pruned x^ stays in a token buffer and the next block reads the kept rows in place
        // (LN1 in the pruning kernel or through the map, the projection's residual through the map).
        // the next block's LN1 folded into its QKV product (its weights carry that form): this block hands over
        // its output tokens themselves with their row sums, whether it drops tokens or not
        const bool fold_next = !last && d->dtype == RS_BF16 && weights[l + 1].w_qkv_ln && weights[l + 1].c_qkv_ln &&
                               weights[l + 1].b_qkv_ln && rs_block_uses_tensor_cores(ctx, &bd);
        const bool in_place = !last && drops[l] > 0 && !taps->x_out[l] && !fold_next && rs_block_uses_tensor_cores(ctx, &bd);
        void* out = in_place ? nullptr : (taps->x_out[l] ? taps->x_out[l] : act[l & 1]);
        // LN1 of block l+1 rides in this block's pruning kernel: one kernel less per block
        const rs::LnFuse next = {last ? nullptr : weights[l + 1].ln1_g, last ? nullptr : weights[l + 1].ln1_b, eps, ln_buf};
        bool ln_done = false;
        // A block that drops nothing hands its output to the next block as it is: if that block's weights
        // carry LN1 folded into QKV, this block's FC2 leaves the row sums and no LN1 kernel runs.
        int parts_out = 0;
        const LoopHooks hk = {cur_map, cur_ln, (last || fold_next || !next.gamma || !next.beta) ? nullptr : &next,
                              in_place ? maps[l & 1] : nullptr, !in_place, &ln_done, nullptr, nullptr, nullptr,
                              cur_stats, cur_parts, fold_next ? stats[l & 1] : nullptr, fold_next ? &parts_out : nullptr};
        rs_status st = block_fwd_impl(ctx, &bd, &weights[l], cur, out, taps->scores ? taps->scores[l] : nullptr,
                                      taps->keep_idx ? taps->keep_idx[l] : nullptr, in_place ? act[l & 1] : nullptr, base,
                                      p.block_ws, stream, &hk);
        if (st != RS_OK) return st;
        cur = in_place ? act[l & 1] : out;
        cur_map = in_place ? maps[l & 1] : nullptr;
        cur_ln = ln_done ? ln_buf : nullptr;
        cur_stats = (fold_next && parts_out > 0) ? stats[l & 1] : nullptr;
        cur_parts = parts_out;
        n -= drops[l];
    }
    return RS_OK;
}

rs_status rs_prepare_ln1_fold(rs_ctx* ctx, rs_dtype dtype, int D, const void* w_qkv, const float* b_qkv,
                              const float* ln1_g, const float* ln1_b, void* w_out, float* c_out, float* b_out,
                              void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!w_qkv || !ln1_g || !ln1_b || !w_out || !c_out || !b_out) return fail(ctx, RS_ERR_INVALID_ARG, "rs_prepare_ln1_fold: null argument");
    if (dtype != RS_BF16 || D < 128 || (D % 128)) return fail(ctx, RS_ERR_UNSUPPORTED, "rs_prepare_ln1_fold: bf16 and D a multiple of 128 only");
    if (!aligned16(w_qkv) || !aligned16(w_out)) return fail(ctx, RS_ERR_INVALID_ARG, "rs_prepare_ln1_fold: misaligned pointer");
    cudaError_t e = rs::launch_ln_fold_prep(w_qkv, b_qkv, ln1_g, ln1_b, 3 * D, D, w_out, c_out, b_out, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "rs_prepare_ln1_fold");
    ctx->launches += 1;
    return RS_OK;
}

rs_status rs_vit_fwd_ragged(rs_ctx* ctx, const rs_vit_desc* d, const rs_block_weights* weights, const int* pad_drops,
                            const void* x, void* x_out, int32_t* keep_last, const int32_t* seq_lens,
                            const int32_t* sample_drops, int32_t* lens_out, void* workspace, size_t workspace_bytes,
                            void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!d || !weights || !pad_drops || !x || !x_out || !seq_lens || !sample_drops || d->L < 1)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_vit_fwd_ragged: null argument");
    VitPlan p;
    if (!valid_dtype(d->dtype) || !vit_plan(*d, pad_drops, &p))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_vit_fwd_ragged: bad descriptor or schedule (need 0 <= pad_drops[l] <= N_l - 1)");
    if (!workspace || workspace_bytes < p.total)
        return fail(ctx, RS_ERR_WORKSPACE, "rs_vit_fwd_ragged: workspace of %zu bytes needed, %zu given", p.total, workspace_bytes);
    if (reinterpret_cast<uintptr_t>(workspace) & 255u)
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_vit_fwd_ragged: workspace must be 256-byte aligned");
    if ((reinterpret_cast<uintptr_t>(seq_lens) & 3u) || (reinterpret_cast<uintptr_t>(sample_drops) & 3u))
        return fail(ctx, RS_ERR_INVALID_ARG, "rs_vit_fwd_ragged: misaligned count arrays");
    char* base = (char*)workspace;
    void* act[2] = {base + p.block_ws, base + p.block_ws + p.act_bytes};
    // the per-sample counts between the blocks live where rs_vit_fwd keeps its row-index lists
    int32_t* lens[2] = {(int32_t*)(base + p.block_ws + 3 * p.act_bytes), (int32_t*)(base + p.block_ws + 3 * p.act_bytes + p.map_bytes)};
    const void* cur = x;
    const int32_t* cur_lens = seq_lens;
    int n = d->N;
    for (int l = 0; l < d->L; ++l) {
        const bool last = l == d->L - 1;
        rs_block_desc bd = {d->dtype, d->dtype, d->B, n, d->D, d->H, d->D_mlp, pad_drops[l], d->has_cls, d->ln_eps, d->scale,
                            d->score_mode, d->dist};
        void* out = last ? x_out : act[l & 1];
        int32_t* next_lens = last ? lens_out : lens[l & 1];
        const LoopHooks hk = {nullptr, nullptr, nullptr, nullptr, true, nullptr, cur_lens, sample_drops + (size_t)l * d->B, next_lens,
                              nullptr, 0, nullptr, nullptr};
        rs_status st = block_fwd_impl(ctx, &bd, &weights[l], cur, out, nullptr, last ? keep_last : nullptr, nullptr, base,
                                      p.block_ws, stream, &hk);
        if (st != RS_OK) return st;
        cur = out;
        cur_lens = next_lens;
        n -= pad_drops[l];
    }
    return RS_OK;
}

rs_status rs_vit_fwd(rs_ctx* ctx, const rs_vit_desc* d, const rs_block_weights* weights, const int* drops,
                     const void* x, void* x_out, float* scores_last, int32_t* keep_last, void* workspace,
                     size_t workspace_bytes, void* stream) {
    if (!ctx) return RS_ERR_INVALID_ARG;
    if (!d || d->L < 1 || d->L > 4096 || !x_out) return fail(ctx, RS_ERR_INVALID_ARG, "rs_vit_fwd: null argument or bad L");
    std::vector<void*> xo(d->L, nullptr);
    std::vector<float*> sc(d->L, nullptr);
    std::vector<int32_t*> ki(d->L, nullptr);
    xo[d->L - 1] = x_out; sc[d->L - 1] = scores_last; ki[d->L - 1] = keep_last;
    const rs_vit_taps taps = {xo.data(), sc.data(), ki.data()};
    return rs_vit_fwd_taps(ctx, d, weights, drops, x, &taps, workspace, workspace_bytes, stream);
}

}  // extern "C"
