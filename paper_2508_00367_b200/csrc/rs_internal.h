// Internal declarations shared by the translation units of the library: the
// context object and the host-side launchers of every kernel.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include <stddef.h>

#include "rs.h"
#include "rs_profile.h"

// Tensor maps are encoded once per (pointer, shape, box) and kept in the context: a block's launches
// name the same few buffers over and over, and every cuTensorMapEncodeTiled call costs about a
// microsecond of host time.  128 slots, eight probed per lookup; a full neighbourhood evicts its home slot.
struct rs_tmap_key {
    const void* base;
    unsigned long long dims[4], strides[3];
    unsigned int box[4];
    unsigned int rank, dtype, swizzle, pad;
};
struct rs_tmap_slot {
    CUtensorMap map;
    rs_tmap_key key;
    int valid;
};
enum { kTmapSlots = 128 };

struct rs_ctx {
    int device;
    int sm_count;
    int use_tc;            // tcgen05 kernels enabled for bf16
    int require_tc;        // RS_REQUIRE_TC=1: a bf16 shape the tensor-core kernels cannot take is an error
    int* d_status;         // device status word (0 = ok), first bytes of a small allocation made by rs_create
    unsigned char* d_flags; // keep-flag scratch of rs_topk_compact (kFlagScratch bytes, same allocation)
    int log, nvtx;          // RS_LOG=1: a line per launch on stderr; RS_NVTX=1: an NVTX range around each launch call
    int attn_kernel;        // RS_ATTN_KERNEL: 0 the faster attention kernel per shape (cost model), 2 / 3 always that one
    long long launches;    // kernels launched through this context
    void* encode_tiled;    // cuTensorMapEncodeTiled entry point (driver API), or null
    int timing;            // bracket launches with events
    int n_events;          // recorded launches since the last read
    cudaEvent_t* ev;       // 2 * kMaxTimed events, created on first enable
    unsigned char* ev_class;
    char err[512];
    long long tmap_hits, tmap_misses;
    rs_tmap_slot tmaps[kTmapSlots];   // (CUtensorMap wants 64-byte alignment: the context is allocated accordingly)
};

enum { kMaxTimed = 8192 };
enum { kFlagScratch = 1 << 20 };

// Device status word values.
enum { RS_DEV_OK = 0, RS_DEV_TIMEOUT = 1, RS_DEV_SMEM_ALIGN = 2 };

namespace rs {

// Launch with programmatic stream serialization: the kernel may begin (up to its grid_dep_wait())
// while the previous kernel of the stream is finishing.  Every kernel launched this way calls
// grid_dep_wait() before it touches global memory.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

inline size_t dtype_size(rs_dtype t) { return t == RS_BF16 ? 2 : 4; }
inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- memory-bound kernels (rs_elementwise.cu) ----
// LayerNorm over the last dimension: x [T, D] (in_dtype) -> out [T, D] (out_dtype); fp32 math.
// row_map (optional, [T] int32): output row t normalises input row row_map[t] instead of row t.
cudaError_t launch_layernorm(rs_dtype in_dtype, rs_dtype out_dtype, const void* x, const float* gamma,
                             const float* beta, float eps, long long T, int D, void* out,
                             const int32_t* row_map, cudaStream_t st);
// s[t] = D(after[t,:], before[t,:]).
cudaError_t launch_shift_score(rs_dtype dtype, rs_dist dist, long long T, int D, const void* after,
                               const void* before, float* scores, cudaStream_t st);
// Residual-add epilogue with the score fused in: x_hat = m + x_prime (out_dtype);
// s = |m - x_prime| (MLP), |m| (MLP_DELTA), |x_prime - 2 x| = |SA(LN(x)) - x| (ATTN) or
// |x_hat - x| (BLOCK).  m, x_prime fp32; x (the block input, x_dtype) only for ATTN and BLOCK.
cudaError_t launch_residual_score(const float* m, const float* x_prime, const void* x, rs_dtype x_dtype,
                                  long long T, int D, rs_score_mode mode, rs_dist dist, rs_dtype out_dtype,
                                  void* x_hat, float* scores, cudaStream_t st);

// ---- selection and compaction (rs_select.cu) ----
// scores: [B, N] fp32; or, if nparts > 0, the per-tile partial sums a GEMM epilogue left
// (nparts = tiles | rs_dist << 16; [B*N, tiles] sums, three per tile for the cosine distance),
// from which the score is finished here (and written to scores_out when non-null).
// row_map (optional, [B, K] int32): flat source row b * N + keep_idx[b, j] of every kept token, with
// which the next block reads the un-pruned rows in place.
// flags / flags_bytes: 4-byte aligned scratch between the flag kernel and the row kernel (a byte
// per token and a count per 64 or 128 tokens; with less than the whole batch needs, the batch is
// processed in several passes, with less than one sample needs the radix kernel runs instead).
// *launches (optional) receives the number of kernels launched.
cudaError_t launch_select(const float* scores, int nparts, float* scores_out, int B, int N, int K,
                          int has_cls, int32_t* keep_idx, int32_t* row_map, uint8_t* flags, size_t flags_bytes,
                          int sm_count, cudaStream_t st, int* launches);
// The compaction kernels can also write LN(x_out) for the block that follows (its LN1 of Eq. att):
// the warp that copies a kept row has it in registers.  out: [B, K, D] of the rows' dtype.
// gamma == null with stats set: no LayerNorm; the kept rows are copied and the sum and sum of squares of each
// copied row's bf16 values go to stats[2 * row], stats[2 * row + 1] (for a LayerNorm folded into the next product).
struct LnFuse { const float* gamma; const float* beta; float eps; void* out; float* stats; };
bool ln_fusable(rs_dtype dtype, int D);   // the row fits the registers of one warp
// x_out may be null when ln is given: only the normalised rows are written (no dense copy).
cudaError_t launch_gather(rs_dtype dtype, const void* x, const int32_t* keep_idx, int B, int N, int K,
                          int D, void* x_out, const LnFuse* ln /*null: none*/, cudaStream_t st);
// Selection, index lists and the rows' move (N <= 4608 and something is dropped): a kernel that finds
// the cut of every sample and flags its kept tokens (a CTA per sample), then a warp per kept row.
// x null: indices only.  x given: x_out (dense copy) and / or ln (normalised rows) must be given.
bool prune_fusable(int N, int K, size_t flags_bytes);
cudaError_t launch_prune(const float* scores, int nparts, float* scores_out, int B, int N, int K, int has_cls,
                         int32_t* keep_idx, int32_t* row_map, rs_dtype dtype, const void* x, int D, void* x_out,
                         const LnFuse* ln /*null: none*/, uint8_t* flags, size_t flags_bytes, int sm_count,
                         cudaStream_t st, int* launches, const int32_t* seq_lens /*dev [B] or null*/,
                         const int32_t* drops /*dev [B], with seq_lens*/, int32_t* lens_out /*dev [B] or null*/);
// Line-wise pruning of a 2-D token grid: keep_rows [B, Hk], keep_cols [B, Wk] and, when x is given,
// x_out[b, i, j, :] = x[b, keep_rows[b, i], keep_cols[b, j], :].  H, W <= linewise_max_lines().
int linewise_max_lines();
cudaError_t launch_linewise(const float* scores, int B, int H, int W, int Hk, int Wk, int32_t* keep_rows,
                            int32_t* keep_cols, rs_dtype dtype, const void* x, int D, void* x_out, int sm_count,
                            cudaStream_t st);
size_t select_smem_bytes(int N);
cudaError_t select_init();   // opt in to large dynamic shared memory, once per device (the current one)

// ---- SIMT contraction path (rs_simt.cu): fp32 FMA, used for RS_F32 and as a cross-check ----
// out[M, N] = act(A[M, K] * W[N, K]^T + bias) + residual.
cudaError_t launch_gemm_simt(rs_dtype in_dtype, const void* A, const void* W, const float* bias,
                             int gelu, const void* residual, rs_dtype res_dtype, void* out,
                             rs_dtype out_dtype, long long M, int N, int K, cudaStream_t st);
cudaError_t launch_attn_simt(const rs_attn_desc& d, const void* q, const void* k, const void* v,
                             void* out, cudaStream_t st);

// ---- tcgen05 GEMM (rs_gemm_tc.cu): bf16 operands, fp32 accumulation in tensor memory ----
enum { RS_EPI_BIAS = 0, RS_EPI_BIAS_GELU = 1, RS_EPI_RESID = 2, RS_EPI_SCORE = 3 };
void* tc_get_encode_fn();                       // cuTensorMapEncodeTiled via the runtime, or null
// Tiled tensor map of `rank` dimensions over bf16 (dtype 0) or fp32 (dtype 1) elements, through the
// context's cache; strides in bytes for dimensions 1 .. rank-1.  False when the driver refuses it.
bool tc_encode_cached(rs_ctx* ctx, CUtensorMap* out, const void* base, int rank, int dtype, const unsigned long long* dims,
                      const unsigned long long* strides, const unsigned int* box, int swizzle_bytes);
bool gemm_tc_supported(long long M, int N, int K);
int gemm_tc_score_parts(const rs_ctx* ctx, long long M, int N);   // partial sums per row written by RS_EPI_SCORE
// out[M, N] = epilogue(A[M, K] . W[N, K]^T); see rs_gemm_tc.cu for the epilogues.
// row_map (optional, [M] int32): row t of the block input (the bf16 residual of RS_EPI_RESID, residual2
// of RS_EPI_SCORE) is row row_map[t] of the given matrix -- the un-pruned output of the previous block.
cudaError_t launch_ln_fold_prep(const void* W, const float* bias, const float* g, const float* beta, int n_out, int K,
                                void* w_out, float* c_out, float* b_out, cudaStream_t st);
// LayerNorm folded across two products (the layer loop's non-pruning blocks): the FC2 launch of a block also
// leaves per-row partial sums (stats_out, and how many per row in *stats_parts_out); the QKV launch of the
// next block reads them (stats_in, stats_parts) and applies the normalisation in its epilogue, with the
// prepared weights of rs_prepare_ln1_fold as W and bias and their column sums c.
struct GemmLn {
    float* stats_out;
    int* stats_parts_out;
    const float* stats_in;
    int stats_parts;
    const float* colsum;
    float eps;
};
cudaError_t launch_gemm_tc(rs_ctx* ctx, int epi, const void* A, const void* W, const float* bias,
                           const void* residual, const void* residual2, const int32_t* row_map, void* out,
                           rs_dtype out_dtype, float* partials, int score_kind, int dist, long long M, int N, int K,
                           cudaStream_t st, const GemmLn* ln = nullptr);

// ---- tcgen05 attention (rs_attn_tc.cu): bf16, head dimension 64 ----
bool attn_tc_supported(const rs_attn_desc& d);
// Which attention kernel runs a shape of BH (sample, head)s and N > 128 tokens on G SMs, and how: best_hs heads handed
// out tile by tile (two-tile kernel), three = the three-tile kernel is expected to be faster, wrap3 its tail placement.
struct AttnPlan { long long best_hs; int three, wrap3; };
AttnPlan attn_plan(long long BH, int N, int G);
// Three query tiles per CTA (rs_attn_tc3.cu), N > 128: the longest CTA's load under its item list, and the launch.
long long attn_tc3_plan(long long BH, int N, int G, int* wrap);
cudaError_t launch_attn_tc3(rs_ctx* ctx, const rs_attn_desc& d, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                            const CUtensorMap& tmV, const CUtensorMap& tmO, int wrap, cudaStream_t st);
// seq_lens (optional, dev [B]): sample b attends over its first seq_lens[b] tokens only.
cudaError_t launch_attn_tc(rs_ctx* ctx, const rs_attn_desc& d, const void* q, const void* k, const void* v,
                           void* out, const int32_t* seq_lens, cudaStream_t st);

}  // namespace rs
