// bf16 GEMM on the 5th-generation tensor cores with the block's epilogues fused in:
//     out[M, N] = epilogue(A[M, K] . W[N, K]^T)
// A and W are K-major.  Two CTAs on neighbouring SMs form a pair (a cluster of two) that owns
// a 256 x BN output tile: each CTA loads its own 128 rows of A and BN/2 rows of W by TMA
// (128-byte swizzle, no multicast) into a shared-memory ring, and one thread of the pair's
// leader issues tcgen05.mma.cta_group::2, which reads both CTAs' shared memory and accumulates
// each CTA's 128 x BN half in that CTA's tensor memory.  Per byte moved from L2 to the SMs the
// pair tile does twice the arithmetic of a 128 x 128 tile, which is what lifts the kernel off
// the L2 -> SM bandwidth bound.  The fp32 accumulator is double-buffered in tensor memory, so
// the eight epilogue warps of each CTA drain tile i (tcgen05.ld -> bias / GELU / residual /
// score -> swizzled shared memory -> one TMA store per warp and 128-byte column block) while the
// main loop of tile i+1 runs.
//
// Epilogues (Eq. att, Eq. MLP, Sec. 3.2):
//   EPI_BIAS       out = acc + b                          -> bf16      (QKV projection)
//   EPI_BIAS_GELU  out = GELU(acc + b)                    -> bf16      (FC1)
//   EPI_RESID      a = acc + b;  out = a + x              -> fp32      (projection + residual = x');
//                  optionally partial sums of (a - x)^2 per row    (shift through attention, choice (i))
//   EPI_SCORE      m = acc + b;  out = m + x';  partial sums of (m - x')^2, m^2 or (out - x)^2 per row
//                                                          -> bf16/fp32 (FC2 + residual + shift score)
#include <string.h>

#include "rs_internal.h"
#include "rs_device.cuh"
#include "rs_once.h"
#include "rs_tc.cuh"

namespace rs {

namespace {

using namespace tc;

// EPI_SCORE_STATS: EPI_SCORE that also leaves, per row and column half of a tile, the sum and the sum of
// squares of the (rounded) output values -- the row statistics of the next block's LayerNorm.
// EPI_BIAS_LN: the LayerNorm of the A operand folded into the product: with W' = W * gamma (column-wise),
// c_n = sum_k W'_nk and b'_n = b_n + sum_k W_nk beta_k,  LN(x) W^T + b = rstd (x W'^T - mu c) + b';  mu and
// rstd of a row come from the statistics above, acc = x W'^T from the tensor cores.
enum { EPI_BIAS = 0, EPI_BIAS_GELU = 1, EPI_RESID = 2, EPI_SCORE = 3, EPI_SCORE_STATS = 4, EPI_BIAS_LN = 5 };

constexpr int BM = 128;                       // rows per CTA; the pair's tile has 2 * BM rows
constexpr int BK = 64;
constexpr int kThreads = 320;                 // warp 0: TMA, warp 1: MMA (leader CTA), warps 2-9: epilogue
constexpr int kEpiWarps = 8;
constexpr int A_BYTES = BM * BK * 2;          // 16 KB
constexpr int STG_BYTES = 32 * 128;           // one staged output block of a warp: its 32 rows of 128 bytes
constexpr int RES_BOX_BYTES = 32 * 64;         // residual of one 32-column chunk of a warp: 32 rows of 32 bf16

// EPI_RESID brings the bf16 residual of a warp's rows in by TMA (a row per lane read straight from
// global memory touches 32 lines per load instruction and cost a fifth of the projection's time):
// one buffer per warp for a whole tile, loaded while the previous tile's main loop runs.  It pays
// for the room with one staging buffer per warp instead of two and one operand stage less.
template <int BN, int EPI> struct Cfg {
    static constexpr bool RES_TMA = EPI == EPI_RESID;
    static constexpr bool LN = EPI == EPI_BIAS_LN;                 // one staging buffer per warp, room for a second column vector
    static constexpr int B_BYTES = (BN / 2) * BK * 2;              // this CTA's half of the W tile
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int STAGES = (BN == 128) ? 6 : RES_TMA ? 4 : 5;
    static constexpr int TMEM_COLS = (BN == 128) ? 256 : 512;      // two accumulators, a power of two
    static constexpr int SPLIT = (BN == 128) ? 64 : 128;           // epilogue warps 2-5 take columns [0, SPLIT)
    static constexpr int STG_PER_WARP = (RES_TMA || LN) ? 1 : 2;
    static constexpr int RES_WARP_BYTES = RES_TMA ? (SPLIT / 32) * RES_BOX_BYTES : 0;   // the wider half's chunks
    static constexpr int OFF_STG = STAGES * STAGE_BYTES;
    static constexpr int OFF_RES = OFF_STG + kEpiWarps * STG_PER_WARP * STG_BYTES;
    static constexpr int OFF_BAR = OFF_RES + kEpiWarps * RES_WARP_BYTES;
    static constexpr int OFF_BIAS = OFF_BAR + 256;                 // float [2 tile parities][2 halves][128]: bias slices
    static constexpr int OFF_COLSUM = OFF_BIAS + 2048;             // EPI_BIAS_LN: float [2][2][128] like the bias slices
    static constexpr size_t SMEM = (size_t)OFF_BIAS + (LN ? 4096 : 2048);   // the window itself must be 1024-byte aligned
    static_assert(SMEM <= 227 * 1024, "shared memory of one CTA");
};

struct GemmArgs {
    int M, N, K;
    const float* bias;        // [N] or null
    const void* residual;     // EPI_RESID: bf16 [M, N];  EPI_SCORE: fp32 [M, N]
    const void* residual2;    // EPI_SCORE, score_kind 2: bf16 [M, N] block input x
    const int* row_map;       // optional [M]: row t of the block input (EPI_RESID's residual, EPI_SCORE's residual2)
                              // is row row_map[t] of that matrix (the previous block's un-pruned output, read in place)
    float* partials;          // EPI_SCORE (and EPI_RESID when non-null): [M, 2 * N / BN] sums of squares
    int score_kind;           // EPI_SCORE: scored pair (u, v) = 0: (m, x'), 1: (x^, x'), 2: (x^, x)
    int dist;                 // rs_dist of the score: L2 / L1 sums of (u - v)^2 / |u - v|, cosine sums of u.v, u.u, v.v
    float* stats_out;         // EPI_SCORE_STATS: [M, 2 * N / BN][2] = (sum, sum of squares) of the row's outputs in that half tile
    const float* stats_in;    // EPI_BIAS_LN: such statistics of the A operand's rows, stats_parts pairs per row over ln_dim = K values
    const float* colsum;      // EPI_BIAS_LN: c [N]
    int stats_parts;
    float ln_eps;
    int* status;
};

// Exact-erf GELU, v * Phi(v), to fp32 accuracy (max abs error 8e-7 over all v) without erff:
// with q(t) = -log2(Phi(-t)) for t >= 0,  Phi(v) = 2^-q(|v|) for v < 0 and 1 - 2^-q(|v|) for
// v >= 0.  q is smooth (about t^2/2 * log2(e) plus slow terms) and a degree-5 polynomial fitted
// on [0, 7] with weight t * Phi(-t) reproduces GELU to that accuracy; its positive leading
// coefficient keeps 2^-q -> 0 for large |v|.  Coefficients from csrc/fit_gelu.py.
__device__ __forceinline__ float gelu_erf(float v) {
    const float a = fabsf(v);
    float q = 0.00047694556997157633f;
    q = fmaf(q, a, -0.00711308466270566f);
    q = fmaf(q, a, 0.05190887302160263f);
    q = fmaf(q, a, 0.4598882496356964f);
    q = fmaf(q, a, 1.1508461236953735f);
    q = fmaf(q, a, 1.0000265836715698f);
    float e;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(-q));
    return v * (v >= 0.f ? 1.f - e : e);
}

// Adds one element of the scored pair (u, v) to the running sums of the chosen distance (Sec. 3.3).
__device__ __forceinline__ void score_acc(int dist, float u, float v, float& s0, float& s1, float& s2) {
    if (dist == RS_DIST_L2) { const float d = u - v; s0 = fmaf(d, d, s0); }
    else if (dist == RS_DIST_L1) { s0 += fabsf(u - v); }
    else { s0 = fmaf(u, v, s0); s1 = fmaf(u, u, s1); s2 = fmaf(v, v, s2); }
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}

template <int BN, int EPI, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmOut, const __grid_constant__ CUtensorMap tmRes,
               const GemmArgs args) {
    using C = Cfg<BN, EPI>;
    // The 128-byte swizzle wants 1024-byte aligned stage and staging buffers, and the layout leaves no
    // room to round the base up: a window that is not aligned is reported, and nothing else is done.
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    uint8_t* smem = smem_raw;
    if (smem_u32(smem) & 1023u) {
        if (threadIdx.x == 0) atomicExch(args.status, RS_DEV_SMEM_ALIGN);
        return;
    }
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + C::OFF_BAR);
    uint64_t* full = bars;                       // [STAGES] leader's: both CTAs' operands landed
    uint64_t* empty = bars + C::STAGES;          // [STAGES] per CTA: the MMAs reading the stage retired
    uint64_t* tfull = bars + 2 * C::STAGES;      // [2] per CTA: accumulator complete
    uint64_t* tempty = bars + 2 * C::STAGES + 2; // [2] leader's: both CTAs' epilogues drained it
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
    volatile int* half_fail = reinterpret_cast<volatile int*>(tmem_slot + 2);   // [2]
    uint64_t* res_full = bars + 2 * C::STAGES + 6;   // [kEpiWarps] the warp's residual of a tile landed (EPI_RESID)

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();     // 0 = leader of the pair
    const int num_m = (args.M + 2 * BM - 1) / (2 * BM), num_n = args.N / BN;
    const int tiles = num_m * num_n, kblocks = args.K / BK;
    const int pair = (int)cluster_id_x(), npairs = (int)cluster_count_x();

    if (threadIdx.x == 0) {
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        prefetch_tmap(&tmOut);
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], 2 * kEpiWarps); }
        if (C::RES_TMA) {
            prefetch_tmap(&tmRes);
            // one arrival by the lane that starts the TMA copies, or one by each lane's own indexed copies
            for (int w = 0; w < kEpiWarps; ++w) mbar_init(&res_full[w], args.row_map ? 32 : 1);
        }
        *abort_flag = 0;
        half_fail[0] = 0;
        half_fail[1] = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(tmem_slot, C::TMEM_COLS);
        tmem_relinquish_pair();
    }
    tc_fence_before();
    __syncthreads();
    cluster_sync();                              // the peer's barriers exist before anything signals them
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above touched no global memory and may overlap the previous kernel's tail.
    grid_dep_launch();
    grid_dep_wait();

    if (warp == 0) {
        // ---------------- TMA producer (both CTAs; each loads its own halves) ----------------
        if (elect_one()) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = pair; tile < tiles && ok; tile += npairs) {
                const int m0 = (tile / num_n) * (2 * BM) + (int)rank * BM;
                const int n0 = (tile % num_n) * BN + (int)rank * (BN / 2);
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t* sa = smem + (size_t)s * C::STAGE_BYTES;
                    const uint32_t lead_full = map_to_cta(smem_u32(&full[s]), 0);
                    if (rank == 0) mbar_expect_tx(&full[s], 2 * C::STAGE_BYTES);
                    tma_load_2d_pair(sa, &tmA, lead_full, kb * BK, m0);
                    tma_load_2d_pair(sa + A_BYTES, &tmB, lead_full, kb * BK, n0);
                }
            }
            // Every stage this thread filled must have been consumed (which implies its copies
            // landed and the leader's commit signals reached this CTA) before the CTA may exit.
            const uint32_t issued = it;
            for (int s = 0; s < C::STAGES && ok; ++s) {
                if ((uint32_t)s >= issued) break;
                const uint32_t last = ((issued - 1 - s) / C::STAGES) * C::STAGES + s;   // last use of stage s
                ok = mbar_wait(&empty[s], (last / C::STAGES) & 1u, abort_flag);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer (leader CTA only) ----------------
        if (rank == 0 && elect_one()) {
            constexpr uint32_t idesc = idesc_bf16(2 * BM, BN, 0, 0);
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int tile = pair; tile < tiles && ok; tile += npairs, ++tl) {
                const uint32_t a = tl & 1u, aph = (tl >> 1) & 1u;
                if (!mbar_wait(&tempty[a], aph ^ 1u, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + a * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    if (!mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = smem_u32(smem + (size_t)s * C::STAGE_BYTES);
                    const uint64_t da = smem_desc_sw128(sa, 16, 1024);
                    const uint64_t db = smem_desc_sw128(sa + A_BYTES, 16, 1024);
#pragma unroll
                    for (int k = 0; k < BK / 16; ++k)   // 32 bytes along K per MMA: +2 in the address field
                        mma_ss_pair(d_tmem, da + 2u * k, db + 2u * k, idesc, (kb | k) != 0);
                    mma_commit_pair(&empty[s], 3);      // frees the stage in both CTAs when these MMAs retire
                }
                if (ok) mma_commit_pair(&tfull[a], 3);  // accumulator complete in both CTAs
            }
        }
    } else {
        // ---------------- epilogue (both CTAs; each drains its own 128 x BN half) ----------------
        const int q = warp & 3;                          // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;                // warps 2-5: columns [0, SPLIT), warps 6-9: the rest
        const int c_begin = half ? C::SPLIT : 0, c_end = half ? BN : C::SPLIT;
        constexpr int BLK_COLS = 128 / (int)sizeof(OutT);            // columns in one staged 128-byte row
        constexpr int CHUNKS_PER_BLK = BLK_COLS / 32;                // 32-column TMEM loads per staged block
        const int trow = q * 32 + lane;                  // row inside this CTA's half of the tile
        const uint32_t stg_row = (uint32_t)(lane >> 3) * 1024u + (uint32_t)(lane & 7) * 128u;   // inside the warp's 32-row slab
        const int r8 = lane & 7;
        const int t128 = ((warp - 2) & 3) * 32 + lane;   // this thread's index among the 128 of its half
        const uint32_t lead_tempty[2] = {map_to_cta(smem_u32(&tempty[0]), 0), map_to_cta(smem_u32(&tempty[1]), 0)};
        uint32_t tl = 0, blk_ctr = 0;
        // EPI_RESID: the residual of this warp's 32 rows x its half's columns of a tile, one 64-byte-
        // swizzled box per 32-column chunk (rows past M arrive as zeros)
        uint8_t* res_buf = smem + C::OFF_RES + (warp - 2) * C::RES_WARP_BYTES;
        auto issue_res = [&](int tile) {
            const int rm0 = (tile / num_n) * (2 * BM) + (int)rank * BM + q * 32, rn0 = (tile % num_n) * BN;
            mbar_expect_tx(&res_full[warp - 2], (uint32_t)((c_end - c_begin) / 32) * RES_BOX_BYTES);
            for (int c = c_begin; c < c_end; c += 32)
                tma_load_2d(res_buf + ((c - c_begin) / 32) * RES_BOX_BYTES, &tmRes, &res_full[warp - 2], rn0 + c, rm0);
        };
        // The same boxes filled row by row through the row map: lane l looks up the source row of the
        // warp's row l; 16-byte asynchronous copies, a row's pieces by neighbouring lanes, land in the
        // layout the tensor map's 64-byte swizzle would give; rows past M are zero-filled.
        auto issue_res_mapped = [&](int tile) {      // whole warp
            const int rm0 = (tile / num_n) * (2 * BM) + (int)rank * BM + q * 32, rn0 = (tile % num_n) * BN;
            const int src_row = rm0 + lane < args.M ? __ldg(args.row_map + rm0 + lane) : -1;
            const int ppr = (c_end - c_begin) / 8, total = 32 * ppr;          // 16-byte pieces per row
            const __nv_bfloat16* base = reinterpret_cast<const __nv_bfloat16*>(args.residual) + rn0 + c_begin;
            for (int idx = lane; idx < total; idx += 32) {
                const int r = idx / ppr, piece = idx - r * ppr;
                const int sr = __shfl_sync(0xffffffffu, src_row, r);
                const uint32_t dst = smem_u32(res_buf + (piece >> 2) * RES_BOX_BYTES + r * 64 + (((piece & 3) ^ ((r >> 1) & 3)) << 4));
                const __nv_bfloat16* src = base + (size_t)(sr < 0 ? 0 : sr) * args.N + piece * 8;
                asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(sr < 0 ? 0 : 16) : "memory");
            }
            asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(smem_u32(&res_full[warp - 2])) : "memory");
        };
        if (C::RES_TMA && pair < tiles) {
            if (args.row_map) issue_res_mapped(pair);
            else if (lane == 0) issue_res(pair);
        }
        constexpr bool SCORE = EPI == EPI_SCORE || EPI == EPI_SCORE_STATS;
        constexpr int RES_VECS = EPI == EPI_RESID ? 4 : SCORE ? 8 : 1;   // 16-byte loads per 32 columns
        // EPI_BIAS_LN: the partial row sums of this thread's row of the NEXT tile are fetched a tile ahead into
        // registers (up to kLnPre pairs; more are read on the spot), so their way from L2 is never waited for
        constexpr int kLnPre = EPI == EPI_BIAS_LN ? 16 : 1;
        float2 ln_pre[kLnPre];
        auto ln_fetch = [&](int tile) {
            const int frow = (tile / num_n) * (2 * BM) + (int)rank * BM + trow;
            const bool ok = tile < tiles && frow < args.M && args.stats_parts <= kLnPre;
            const float2* sp = reinterpret_cast<const float2*>(args.stats_in) + (size_t)(ok ? frow : 0) * args.stats_parts;
#pragma unroll
            for (int p = 0; p < kLnPre; ++p) ln_pre[p] = (ok && p < args.stats_parts) ? __ldg(sp + p) : make_float2(0.f, 0.f);
        };
        if (EPI == EPI_BIAS_LN) ln_fetch(pair);
        for (int tile = pair; tile < tiles; tile += npairs, ++tl) {
            const int m0 = (tile / num_n) * (2 * BM) + (int)rank * BM, nt = tile % num_n, n0 = nt * BN;
            const uint32_t a = tl & 1u, aph = (tl >> 1) & 1u;
            const int row = m0 + trow;
            const bool valid = row < args.M;
            // row of the block input x (EPI_SCORE, whole-block shift), possibly through the row map
            const int xrow = (SCORE && args.score_kind == 2 && args.row_map && valid) ? __ldg(args.row_map + row) : row;
            // Residual values of 32 columns of this thread's row (zeros for rows past M).  They are
            // fetched one chunk ahead, the first chunk before the accumulator is even complete.
            auto load_res = [&](int c, uint4* dst) {
                if (SCORE) {
                    const size_t off = (size_t)row * args.N + n0 + c;
                    const uint4* rp = reinterpret_cast<const uint4*>(reinterpret_cast<const float*>(args.residual) + off);
#pragma unroll
                    for (int j = 0; j < RES_VECS; ++j) dst[j] = valid ? __ldg(rp + j) : make_uint4(0u, 0u, 0u, 0u);
                }
            };
            uint4 res_next[RES_VECS];
            load_res(c_begin, res_next);
            // EPI_BIAS_LN: mean and reciprocal standard deviation of this thread's row of A from the partial
            // sums its producer left (fetched while the accumulator is still being computed)
            float ln_mu = 0.f, ln_rstd = 0.f;
            if (EPI == EPI_BIAS_LN) {
                float s1 = 0.f, s2 = 0.f;
                if (args.stats_parts <= kLnPre) {
#pragma unroll
                    for (int p = 0; p < kLnPre; ++p) { s1 += ln_pre[p].x; s2 += ln_pre[p].y; }
                    ln_fetch(tile + npairs);
                } else if (valid) {
                    const float2* sp = reinterpret_cast<const float2*>(args.stats_in) + (size_t)row * args.stats_parts;
                    for (int p = 0; p < args.stats_parts; ++p) {
                        const float2 t = __ldg(sp + p);
                        s1 += t.x; s2 += t.y;
                    }
                }
                const float inv_d = 1.f / (float)args.K;
                ln_mu = s1 * inv_d;
                ln_rstd = rsqrtf(fmaxf(s2 * inv_d - ln_mu * ln_mu, 0.f) + args.ln_eps);
            }
            float st1 = 0.f, st2 = 0.f;                  // EPI_SCORE_STATS: sums over this thread's columns
            // The four warps of a column half decide together whether to go on: the named
            // barriers below have no time limit, so no warp may leave the loop alone.
            // this half's slice of the bias goes to shared memory while the accumulator is still being
            // computed (the barrier below publishes it): the chunk loop then has no global read on its chain.
            // Two copies, by tile parity: a warp may still be reading the last tile's slice.
            float* bias_s = reinterpret_cast<float*>(smem + C::OFF_BIAS) + (tl & 1u) * 256 + half * 128;
            if (c_begin + t128 < c_end) bias_s[t128] = args.bias ? __ldg(args.bias + n0 + c_begin + t128) : 0.f;
            float* cs_s = reinterpret_cast<float*>(smem + C::OFF_COLSUM) + (tl & 1u) * 256 + half * 128;   // EPI_BIAS_LN only
            if (EPI == EPI_BIAS_LN && c_begin + t128 < c_end) cs_s[t128] = __ldg(args.colsum + n0 + c_begin + t128);
            if (!__all_sync(0xffffffffu, mbar_wait(&tfull[a], aph, abort_flag))) half_fail[half] = 1;
            if (C::RES_TMA && !__all_sync(0xffffffffu, mbar_wait(&res_full[warp - 2], tl & 1u, abort_flag))) half_fail[half] = 1;
            named_barrier(1 + half, 128);
            if (half_fail[half]) break;
            tc_fence_after();
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN;
            float sq = 0.f, sq1 = 0.f, sq2 = 0.f;
#pragma unroll 1
            for (int c = c_begin; c < c_end; c += 32) {
                const int cb = (c / 32) % CHUNKS_PER_BLK;            // chunk inside the staged block
                uint8_t* stg = smem + C::OFF_STG + ((warp - 2) * C::STG_PER_WARP + (C::STG_PER_WARP == 2 ? (blk_ctr & 1u) : 0u)) * STG_BYTES;
                if (cb == 0) {
                    // the store that last read this buffer (two blocks ago, or the last one) must be done with it
                    if (lane == 0) tma_store_wait_read<C::STG_PER_WARP - 1>();
                    __syncwarp();
                }
                uint4 res[RES_VECS];
                if (C::RES_TMA) {
                    // this lane's row of the chunk's box: 64 bytes, 16-byte pieces XOR-ed with address bits 7-8
                    const uint8_t* rrow = res_buf + ((c - c_begin) / 32) * RES_BOX_BYTES + lane * 64;
#pragma unroll
                    for (int j = 0; j < RES_VECS; ++j)
                        res[j] = *reinterpret_cast<const uint4*>(rrow + ((j ^ ((lane >> 1) & 3)) << 4));
                } else {
#pragma unroll
                    for (int j = 0; j < RES_VECS; ++j) res[j] = res_next[j];
                    if (c + 32 < c_end) load_res(c + 32, res_next);
                }
                uint32_t r[32];
                __syncwarp();                            // tcgen05.ld is warp-collective
                tmem_ld_32x32(taddr + c, r);
                tmem_wait_ld();
                if (c + 32 >= c_end) {                   // accumulator fully read by this warp
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(lead_tempty[a]);
                }
                const int col = n0 + c;
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    const float4 b = *reinterpret_cast<const float4*>(bias_s + (c - c_begin) + j);
                    if (EPI == EPI_BIAS_LN) {
                        const float4 cc = *reinterpret_cast<const float4*>(cs_s + (c - c_begin) + j);
                        v[j] = fmaf(ln_rstd, fmaf(-ln_mu, cc.x, __uint_as_float(r[j])), b.x);
                        v[j + 1] = fmaf(ln_rstd, fmaf(-ln_mu, cc.y, __uint_as_float(r[j + 1])), b.y);
                        v[j + 2] = fmaf(ln_rstd, fmaf(-ln_mu, cc.z, __uint_as_float(r[j + 2])), b.z);
                        v[j + 3] = fmaf(ln_rstd, fmaf(-ln_mu, cc.w, __uint_as_float(r[j + 3])), b.w);
                    } else {
                        v[j] = __uint_as_float(r[j]) + b.x;
                        v[j + 1] = __uint_as_float(r[j + 1]) + b.y;
                        v[j + 2] = __uint_as_float(r[j + 2]) + b.z;
                        v[j + 3] = __uint_as_float(r[j + 3]) + b.w;
                    }
                }
                if (EPI == EPI_BIAS_GELU) {
#pragma unroll
                    for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
                } else if (EPI == EPI_RESID) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint32_t w[4] = {res[j].x, res[j].y, res[j].z, res[j].w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float x0 = __uint_as_float(w[e] << 16), x1 = __uint_as_float(w[e] & 0xffff0000u);
                            if (args.partials) {                      // (u, v) = (SA(LN(x)), x)
                                score_acc(args.dist, v[8 * j + 2 * e], x0, sq, sq1, sq2);
                                score_acc(args.dist, v[8 * j + 2 * e + 1], x1, sq, sq1, sq2);
                            }
                            v[8 * j + 2 * e] += x0;
                            v[8 * j + 2 * e + 1] += x1;
                        }
                    }
                } else if (SCORE) {
                    if (args.score_kind == 2) {
                        // whole-block shift: x^ - x, with the block input x read here (rows past M: zeros)
                        const uint4* x0p = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(args.residual2) +
                                                                          (size_t)xrow * args.N + col);
#pragma unroll
                        for (int j = 0; j < 4; ++j) {
                            const uint4 xv = valid ? __ldg(x0p + j) : make_uint4(0u, 0u, 0u, 0u);
                            const uint32_t w[4] = {xv.x, xv.y, xv.z, xv.w};
                            const float xp[8] = {__uint_as_float(res[2 * j].x), __uint_as_float(res[2 * j].y),
                                                 __uint_as_float(res[2 * j].z), __uint_as_float(res[2 * j].w),
                                                 __uint_as_float(res[2 * j + 1].x), __uint_as_float(res[2 * j + 1].y),
                                                 __uint_as_float(res[2 * j + 1].z), __uint_as_float(res[2 * j + 1].w)};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float xa = __uint_as_float(w[e] << 16), xb = __uint_as_float(w[e] & 0xffff0000u);
                                const float ya = v[8 * j + 2 * e] + xp[2 * e], yb = v[8 * j + 2 * e + 1] + xp[2 * e + 1];
                                score_acc(args.dist, ya, xa, sq, sq1, sq2);
                                score_acc(args.dist, yb, xb, sq, sq1, sq2);
                                v[8 * j + 2 * e] = ya;
                                v[8 * j + 2 * e + 1] = yb;
                            }
                        }
                    } else {
#pragma unroll
                        for (int j = 0; j < 8; ++j) {
                            const float xs[4] = {__uint_as_float(res[j].x), __uint_as_float(res[j].y),
                                                 __uint_as_float(res[j].z), __uint_as_float(res[j].w)};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float m = v[4 * j + e], y = m + xs[e];
                                score_acc(args.dist, args.score_kind ? y : m, xs[e], sq, sq1, sq2);
                                v[4 * j + e] = y;
                            }
                        }
                    }
                }
                // stage the 32 values of this row: 16-byte pieces, XOR-swizzled like the TMA box
                if (sizeof(OutT) == 2) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        const int piece = cb * 4 + g;
                        const uint4 pk = make_uint4(pack_bf16(v[8 * g], v[8 * g + 1]), pack_bf16(v[8 * g + 2], v[8 * g + 3]),
                                                    pack_bf16(v[8 * g + 4], v[8 * g + 5]), pack_bf16(v[8 * g + 6], v[8 * g + 7]));
                        *reinterpret_cast<uint4*>(stg + stg_row + ((piece ^ r8) << 4)) = pk;
                        if (EPI == EPI_SCORE_STATS) {
                            // the statistics are those of the values as stored: the next block reads these bf16 numbers
                            const uint32_t w[4] = {pk.x, pk.y, pk.z, pk.w};
#pragma unroll
                            for (int e = 0; e < 4; ++e) {
                                const float y0 = __uint_as_float(w[e] << 16), y1 = __uint_as_float(w[e] & 0xffff0000u);
                                st1 += y0 + y1;
                                st2 = fmaf(y0, y0, fmaf(y1, y1, st2));
                            }
                        }
                    }
                } else {
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        *reinterpret_cast<float4*>(stg + stg_row + ((g ^ r8) << 4)) =
                            make_float4(v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                }
                if (cb == CHUNKS_PER_BLK - 1) {
                    // Every warp stores its own 32 rows: no barrier between the warps of a tile.
                    fence_async_smem();                  // staged data visible to the TMA engine
                    __syncwarp();
                    if (lane == 0) {
                        if (m0 + q * 32 < args.M)        // rows past M are dropped by the tensor map's bounds
                            tma_store_2d(&tmOut, stg, col + 32 - BLK_COLS, m0 + q * 32);
                        tma_store_commit();
                    }
                    ++blk_ctr;
                }
            }
            if (C::RES_TMA) {
                __syncwarp();                            // every lane has read its residual rows
                if (tile + npairs < tiles) {
                    if (args.row_map) issue_res_mapped(tile + npairs);
                    else if (lane == 0) issue_res(tile + npairs);
                }
            }
            if (EPI == EPI_SCORE_STATS && valid) {
                const size_t pi = (size_t)row * (2 * num_n) + 2 * nt + half;
                reinterpret_cast<float2*>(args.stats_out)[pi] = make_float2(st1, st2);
            }
            if ((SCORE || (EPI == EPI_RESID && args.partials)) && valid) {
                const size_t pi = (size_t)row * (2 * num_n) + 2 * nt + half;
                if (args.dist == RS_DIST_COS) {
                    args.partials[3 * pi] = sq; args.partials[3 * pi + 1] = sq1; args.partials[3 * pi + 2] = sq2;
                } else {
                    args.partials[pi] = sq;
                }
            }
        }
        if (lane == 0) tma_store_wait<0>();              // all output written before the CTA exits
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicExch(args.status, RS_DEV_TIMEOUT);
    cluster_sync();                                      // neither CTA of the pair leaves while the other may signal it
    if (warp == 1) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, C::TMEM_COLS);
    }
}

// Tensor map over a row-major matrix [rows, cols] (cols contiguous) of 2- or 4-byte elements,
// box [box_rows, 128 bytes of columns], 128-byte swizzle.
bool make_tmap_2d(rs_ctx* ctx, CUtensorMap* out, const void* base, int elem_bytes, uint64_t rows, uint64_t cols,
                  uint32_t box_rows) {
    const unsigned long long dims[2] = {cols, rows}, strides[1] = {cols * (uint64_t)elem_bytes};
    const unsigned int box[2] = {(unsigned int)(128 / elem_bytes), box_rows};
    return tc_encode_cached(ctx, out, base, 2, elem_bytes == 2 ? 0 : 1, dims, strides, box, 128);
}

// Tensor map over the bf16 residual [rows, cols] of the projection: box [32 rows, 32 columns = 64 bytes],
// 64-byte swizzle, zeros for rows past the matrix.
bool make_tmap_res(rs_ctx* ctx, CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols) {
    const unsigned long long dims[2] = {cols, rows}, strides[1] = {cols * 2};
    const unsigned int box[2] = {32, 32};
    return tc_encode_cached(ctx, out, base, 2, 0, dims, strides, box, 64);
}

template <int BN, int EPI, typename OutT>
cudaError_t launch_one(const CUtensorMap& tmA, const CUtensorMap& tmB, const CUtensorMap& tmOut, const CUtensorMap& tmRes,
                       const GemmArgs& args, int sm_count, cudaStream_t st) {
    using C = Cfg<BN, EPI>;
    static PerDeviceOnce attr_once;   // per instantiation: the attribute is per function and per device
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = (cudaError_t)attr_once.run(dev, [] {
        return (int)cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI, OutT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::SMEM);
    });
    if (e != cudaSuccess) return e;
    const int tiles = ((args.M + 2 * BM - 1) / (2 * BM)) * (args.N / BN);
    const int pairs = tiles < sm_count / 2 ? tiles : sm_count / 2;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs, 1, 1);
    cfg.blockDim = dim3(kThreads, 1, 1);
    cfg.dynamicSmemBytes = C::SMEM;
    cfg.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 2;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;   // see grid_dep_wait() in the kernel
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, gemm_tc_kernel<BN, EPI, OutT>, tmA, tmB, tmOut, tmRes, args);
}

// Tile width (256, 192 or 128 columns per pair): the one whose waves over the SM pairs cost
// least, a wave of narrower tiles being charged a little more per column because it moves
// more operand bytes per FLOP.
int pick_bn(long long M, int N, int sm_count) {
    const long long pairs = sm_count / 2, mt = (M + 2 * BM - 1) / (2 * BM);
    const int widths[3] = {256, 192, 128};
    const int penalty[3] = {100, 110, 116};
    int best = 128;
    long long best_cost = -1;
    for (int i = 0; i < 3; ++i) {
        if (N % widths[i]) continue;
        const long long waves = (mt * (N / widths[i]) + pairs - 1) / pairs;
        const long long cost = waves * widths[i] * penalty[i];
        if (best_cost < 0 || cost < best_cost) { best_cost = cost; best = widths[i]; }
    }
    return best;
}

}  // namespace

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

bool tc_encode_cached(rs_ctx* ctx, CUtensorMap* out, const void* base, int rank, int dtype, const unsigned long long* dims,
                      const unsigned long long* strides, const unsigned int* box, int swizzle_bytes) {
    if (!ctx->encode_tiled || rank < 2 || rank > 4) return false;
    rs_tmap_key key;
    memset(&key, 0, sizeof(key));
    key.base = base; key.rank = (unsigned)rank; key.dtype = (unsigned)dtype; key.swizzle = (unsigned)swizzle_bytes;
    for (int i = 0; i < rank; ++i) { key.dims[i] = dims[i]; key.box[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) key.strides[i] = strides[i];
    unsigned long long h = (unsigned long long)(uintptr_t)base * 0x9E3779B97F4A7C15ull;
    for (int i = 0; i < rank; ++i) h = (h ^ key.dims[i] ^ ((unsigned long long)key.box[i] << 40)) * 0x9E3779B97F4A7C15ull;
    h ^= (unsigned long long)swizzle_bytes << 8 | (unsigned long long)dtype;
    // eight neighbouring slots are probed; a new map takes the first free one of them, else the home slot
    const unsigned home = (unsigned)((h >> 32) % kTmapSlots);
    rs_tmap_slot* free_slot = nullptr;
    for (unsigned pr = 0; pr < 8; ++pr) {
        rs_tmap_slot& c = ctx->tmaps[(home + pr) % kTmapSlots];
        if (c.valid && memcmp(&c.key, &key, sizeof(key)) == 0) {
            *out = c.map;
            ctx->tmap_hits += 1;
            return true;
        }
        if (!c.valid && !free_slot) free_slot = &c;
    }
    rs_tmap_slot& slot = free_slot ? *free_slot : ctx->tmaps[home];
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(ctx->encode_tiled);
    cuuint64_t d[4], st[3];
    cuuint32_t bx[4], estr[4] = {1, 1, 1, 1};
    for (int i = 0; i < rank; ++i) { d[i] = dims[i]; bx[i] = box[i]; }
    for (int i = 0; i + 1 < rank; ++i) st[i] = strides[i];
    const CUtensorMapSwizzle sw = swizzle_bytes == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : swizzle_bytes == 64 ? CU_TENSOR_MAP_SWIZZLE_64B
                                                                                                         : CU_TENSOR_MAP_SWIZZLE_NONE;
    CUtensorMap m;
    if (fn(&m, dtype == 0 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, (cuuint32_t)rank,
           const_cast<void*>(base), d, st, bx, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, sw, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
           CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
        return false;
    slot.map = m; slot.key = key; slot.valid = 1;
    ctx->tmap_misses += 1;
    *out = m;
    return true;
}

void* tc_get_encode_fn() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
        return nullptr;
    return fn;
}

bool gemm_tc_supported(long long M, int N, int K) {
    return M >= 1 && M < (1ll << 31) && N >= 128 && (N % 128) == 0 && K >= 64 && (K % 64) == 0;
}

int gemm_tc_score_parts(const rs_ctx* ctx, long long M, int N) {
    return 2 * (N / pick_bn(M, N, ctx->sm_count));
}

cudaError_t launch_gemm_tc(rs_ctx* ctx, int epi, const void* A, const void* W, const float* bias,
                           const void* residual, const void* residual2, const int32_t* row_map, void* out, rs_dtype out_dtype,
                           float* partials, int score_kind, int dist, long long M, int N, int K, cudaStream_t st,
                           const GemmLn* ln) {
    if (!ctx->encode_tiled) return cudaErrorNotSupported;
    if (ln && epi == EPI_SCORE && ln->stats_out && out_dtype == RS_BF16) epi = EPI_SCORE_STATS;
    if (ln && epi == EPI_BIAS && ln->stats_in) epi = EPI_BIAS_LN;
    const int bn = pick_bn(M, N, ctx->sm_count);
    const int out_bytes = (epi == EPI_RESID || (epi == EPI_SCORE && out_dtype == RS_F32)) ? 4 : 2;
    if (epi == EPI_SCORE_STATS && ln->stats_parts_out) *ln->stats_parts_out = 2 * (N / bn);
    CUtensorMap tmA, tmB, tmOut, tmRes;
    if (epi == EPI_RESID && !row_map && !make_tmap_res(ctx, &tmRes, residual, (uint64_t)M, (uint64_t)N)) return cudaErrorInvalidValue;
    if (!make_tmap_2d(ctx, &tmA, A, 2, (uint64_t)M, (uint64_t)K, BM) ||
        !make_tmap_2d(ctx, &tmB, W, 2, (uint64_t)N, (uint64_t)K, (uint32_t)(bn / 2)) ||
        !make_tmap_2d(ctx, &tmOut, out, out_bytes, (uint64_t)M, (uint64_t)N, 32))
        return cudaErrorInvalidValue;
    if (epi != EPI_RESID || row_map) tmRes = tmOut;  // unused by the other epilogues and by the mapped residual
    GemmArgs args;
    args.M = (int)M; args.N = N; args.K = K; args.bias = bias; args.residual = residual;
    args.residual2 = residual2; args.row_map = row_map; args.partials = partials; args.score_kind = score_kind; args.dist = dist; args.status = ctx->d_status;
    args.stats_out = ln ? ln->stats_out : nullptr;
    args.stats_in = ln ? ln->stats_in : nullptr;
    args.colsum = ln ? ln->colsum : nullptr;
    args.stats_parts = ln ? ln->stats_parts : 0;
    args.ln_eps = ln ? ln->eps : 0.f;
    const int sms = ctx->sm_count;
#define RS_GEMM_CASE(E, T)                                                                       \
    return bn == 256   ? launch_one<256, E, T>(tmA, tmB, tmOut, tmRes, args, sms, st)           \
           : bn == 192 ? launch_one<192, E, T>(tmA, tmB, tmOut, tmRes, args, sms, st)           \
                       : launch_one<128, E, T>(tmA, tmB, tmOut, tmRes, args, sms, st)
    switch (epi) {
        case EPI_BIAS: RS_GEMM_CASE(EPI_BIAS, __nv_bfloat16);
        case EPI_BIAS_GELU: RS_GEMM_CASE(EPI_BIAS_GELU, __nv_bfloat16);
        case EPI_RESID: RS_GEMM_CASE(EPI_RESID, float);
        case EPI_SCORE:
            if (out_dtype == RS_F32) RS_GEMM_CASE(EPI_SCORE, float);
            RS_GEMM_CASE(EPI_SCORE, __nv_bfloat16);
        case EPI_SCORE_STATS: RS_GEMM_CASE(EPI_SCORE_STATS, __nv_bfloat16);
        case EPI_BIAS_LN: RS_GEMM_CASE(EPI_BIAS_LN, __nv_bfloat16);
    }
#undef RS_GEMM_CASE
    return cudaErrorInvalidValue;
}

}  // namespace rs
