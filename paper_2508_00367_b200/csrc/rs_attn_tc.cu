// Fused attention on the tensor cores (Eq. sa): out = Softmax(Q K^T * scale) V per
// (sample, head), head dimension 64, without ever writing the N x N matrix.
//
// One CTA owns two 128-row query tiles (A and B) of one (sample, head) and streams the
// keys/values in tiles of 128 through a TMA ring that both query tiles share.  For each
// query tile and key tile:  S = Q K^T (tcgen05.mma, fp32 in tensor memory)  ->  one softmax
// warpgroup (a row per thread) pulls the S row into registers and at once hands the S
// columns back, so the next Q K^T is computed while this tile's exponentials run; it keeps a
// running maximum and sum and writes P = exp2(S*c - m*c) as bf16 into its own tensor-memory
// columns  ->  O += P V (tcgen05.mma with P as the tensor-memory A operand and the V tile as
// an MN-major shared-memory B operand).  The exponentials (MUFU) bound this head dimension,
// so everything else is arranged to keep them flowing: the exponent of a tile is taken
// against the maximum known *before* the tile, in the same pass that finds the tile's own
// maximum; only if that exceeds the running one by more than 2^8 (P would leave bf16's
// comfortable range) is the running maximum raised, O rescaled and the pass repeated.  The
// final division by the row sum makes the result the exact softmax either way.
#include <math.h>

#include "rs_internal.h"
#include "rs_tc.cuh"

namespace rs {

namespace {

using namespace tc;

constexpr int BQ = 128, BKV = 128, DH = 64;
constexpr int TILE_BYTES = 128 * DH * 2;        // 16 KB: a [128, 64] bf16 tile
constexpr int NS = 4;                           // K/V ring stages
constexpr int kThreads = 384;                   // warps 0-3 / 4-7: softmax of tile A / B, warp 8: TMA, warp 9: MMA
constexpr int kSoftmaxRegs = 224, kOtherRegs = 56;   // per-thread register budgets after the warpgroups re-split the pool
constexpr int kTmemCols = 512;                  // S_A 0..127, S_B 128..255, P_A 256..319, P_B 320..383, O_A 384..447, O_B 448..511
constexpr int kPCol = 256, kOCol = 384;
constexpr bool kPingPong = true;
constexpr int kPingPongTiles = 1;
constexpr float kRescaleGap = 8.f;              // log2 units the tile maximum may exceed the running one
// shared memory: Q_A | Q_B | K[NS] | V[NS] | barriers
constexpr int OFF_Q = 0, OFF_K = 2 * TILE_BYTES, OFF_V = (2 + NS) * TILE_BYTES;
constexpr int OFF_BAR = (2 + 2 * NS) * TILE_BYTES;
constexpr size_t kSmem = (size_t)OFF_BAR + 256 + 1024 /*alignment slack*/;

struct AttnArgs {
    __nv_bfloat16* out;      // [B, N, H*64]
    int N, H;
    float scale_log2;        // scale * log2(e)
    int* status;
};

__device__ __forceinline__ float ex2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
// bf16 pair of two non-negative floats with integer instructions only (round half up: add half
// an ulp to the bit patterns, keep the upper halves).  The conversion instruction shares the
// MUFU pipe with the exponentials, which is the pipe this kernel is bound by; this does not.
// Differs from round-to-nearest-even only on exact ties.
__device__ __forceinline__ uint32_t pack_bf16_pos(float a, float b) {
    return __byte_perm(__float_as_uint(a) + 0x8000u, __float_as_uint(b) + 0x8000u, 0x7632);
}

__device__ __forceinline__ float max3(float a, float b, float c) {
    float r;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(r) : "f"(a), "f"(b), "f"(c));
    return r;
}

// Packed fp32 pairs (two lanes of arithmetic per instruction on sm_100).
__device__ __forceinline__ uint64_t pack2(float a, float b) {
    uint64_t r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
    return r;
}
__device__ __forceinline__ void unpack2(uint64_t v, float& a, float& b) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ uint64_t ffma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ uint64_t fadd2(uint64_t a, uint64_t b) {
    uint64_t r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}

// Maximum of a row of S held in registers (valid keys only).
template <bool MASKED>
__device__ __forceinline__ float row_max(const uint32_t (&r)[128], int valid) {
    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
    for (int i = 0; i < 128; i += 4) {
        float a = __uint_as_float(r[i]), b = __uint_as_float(r[i + 1]);
        float c = __uint_as_float(r[i + 2]), d = __uint_as_float(r[i + 3]);
        if (MASKED) {
            if (i >= valid) a = -INFINITY;
            if (i + 1 >= valid) b = -INFINITY;
            if (i + 2 >= valid) c = -INFINITY;
            if (i + 3 >= valid) d = -INFINITY;
        }
        m0 = max3(m0, a, b);
        m1 = max3(m1, c, d);
    }
    return fmaxf(m0, m1);
}

// p_i = exp2(s_i * sl + mneg) for the valid keys (0 for the rest), packed to bf16 pairs in
// place (r[0..63] on return); returns the sum of the unrounded p_i.
template <bool MASKED>
__device__ __forceinline__ float exp_pass(uint32_t (&r)[128], float sl, float mneg, int valid) {
    const uint64_t sl2 = pack2(sl, sl), mneg2 = pack2(mneg, mneg);
    uint64_t l01 = pack2(0.f, 0.f), l23 = l01;
#pragma unroll
    for (int i = 0; i < 128; i += 4) {
        float x0, x1, x2, x3;
        unpack2(ffma2(pack2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sl2, mneg2), x0, x1);
        unpack2(ffma2(pack2(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])), sl2, mneg2), x2, x3);
        if (MASKED) {
            if (i >= valid) x0 = -INFINITY;
            if (i + 1 >= valid) x1 = -INFINITY;
            if (i + 2 >= valid) x2 = -INFINITY;
            if (i + 3 >= valid) x3 = -INFINITY;
        }
        const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);   // ex2(-inf) = 0
        l01 = fadd2(l01, pack2(p0, p1));
        l23 = fadd2(l23, pack2(p2, p3));
        r[i >> 1] = pack_bf16(p0, p1);
        r[(i >> 1) + 1] = pack_bf16(p2, p3);
    }
    float a, b, c, d;
    unpack2(l01, a, b);
    unpack2(l23, c, d);
    return (a + b) + (c + d);
}

__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const AttnArgs args) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint64_t* q_full = bars;                 // Q tiles landed
    uint64_t* k_full = bars + 1;             // [NS] K tile landed
    uint64_t* v_full = bars + 1 + NS;        // [NS] V tile landed
    uint64_t* kv_empty = bars + 1 + 2 * NS;  // [NS] every MMA reading the stage retired
    uint64_t* s_full = bars + 1 + 3 * NS;    // [2] S of tile A / B complete in tensor memory
    uint64_t* p_ready = s_full + 2;          // [2] P written (one arrival per softmax warp)
    uint64_t* o_done = s_full + 4;           // [2] O += P V retired
    uint64_t* s_free = s_full + 6;           // [2] S row in registers, columns reusable (one arrival per warp)
    uint64_t* turn = s_full + 8;             // [2][4] exponent pass of tile A / B, warp q, finished
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_full + 16);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int N = args.N;
    const int q0 = blockIdx.x * (2 * BQ), h = blockIdx.y, b = blockIdx.z;
    const int nkv = (N + BKV - 1) / BKV;
    const bool has_b = q0 + BQ < N;          // the second query tile has at least one row

    if (threadIdx.x == 0) {
        prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV);
        mbar_init(q_full, 1);
        for (int s = 0; s < NS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&v_full[s], 1); mbar_init(&kv_empty[s], 1); }
        for (int g = 0; g < 2; ++g) { mbar_init(&s_full[g], 1); mbar_init(&p_ready[g], 4); mbar_init(&o_done[g], 1); mbar_init(&s_free[g], 4); }
        for (int i = 0; i < 8; ++i) mbar_init(&turn[i], 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 9) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // The third warpgroup (TMA, MMA and two idle warps) hands most of its registers to the
    // two softmax warpgroups, which hold a whole 128-column row of S per thread.
    if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
    if (warp == 8) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            mbar_expect_tx(q_full, has_b ? 2 * TILE_BYTES : TILE_BYTES);
            tma_load_4d(smem + OFF_Q, &tmQ, q_full, 0, h, q0, b);
            if (has_b) tma_load_4d(smem + OFF_Q + TILE_BYTES, &tmQ, q_full, 0, h, q0 + BQ, b);
            int issued = 0;
            bool ok = true;
            for (int j = 0; j < nkv; ++j, ++issued) {
                const int s = j % NS;
                if (!mbar_wait(&kv_empty[s], ((j / NS) & 1) ^ 1, abort_flag)) { ok = false; break; }
                mbar_expect_tx(&k_full[s], TILE_BYTES);
                tma_load_4d(smem + OFF_K + s * TILE_BYTES, &tmK, &k_full[s], 0, h, j * BKV, b);
                mbar_expect_tx(&v_full[s], TILE_BYTES);
                tma_load_4d(smem + OFF_V + s * TILE_BYTES, &tmV, &v_full[s], 0, h, j * BKV, b);
            }
            // every copy started here must have landed before the CTA exits
            if (ok) ok = mbar_wait(q_full, 0, abort_flag);
            for (int s = 0; s < NS && s < issued && ok; ++s) {
                const int last = ((issued - 1 - s) / NS) * NS + s;
                ok = mbar_wait(&k_full[s], (last / NS) & 1, abort_flag) && mbar_wait(&v_full[s], (last / NS) & 1, abort_flag);
            }
        }
    } else if (warp == 9) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            bool ok = mbar_wait(q_full, 0, abort_flag);
            tc_fence_after();
            const uint32_t idesc_o = idesc_bf16(BQ, DH, 0, 1);
            // S_g = Q_g K_j^T : both operands K-major (head dimension contiguous)
            auto issue_s = [&](int g, int j) {
                const int s = j % NS;
                const int valid = min(BKV, N - j * BKV);
                const uint32_t idesc_s = idesc_bf16(BQ, (valid + 15) & ~15, 0, 0);
                const uint64_t dq = smem_desc_sw128(smem_u32(smem + OFF_Q + g * TILE_BYTES), 16, 1024);
                const uint64_t dk = smem_desc_sw128(smem_u32(smem + OFF_K + s * TILE_BYTES), 16, 1024);
#pragma unroll
                for (int k = 0; k < DH / 16; ++k)
                    mma_ss(tmem_base + g * BKV, dq + 2u * k, dk + 2u * k, idesc_s, k != 0);
                mma_commit(&s_full[g]);
            };
            // O_g += P_g V_j : P from tensor memory (bf16 pairs, 8 columns per 16 keys), V MN-major
            // (head dimension contiguous), 16 keys = 2048 bytes per slab.
            auto issue_pv = [&](int g, int j) {
                const int s = j % NS;
                const int valid = min(BKV, N - j * BKV);
                const int ksteps = (valid + 15) >> 4;
                const uint32_t sv = smem_u32(smem + OFF_V + s * TILE_BYTES);
                for (int k = 0; k < ksteps; ++k)
                    mma_ts(tmem_base + kOCol + g * DH, tmem_base + kPCol + g * DH + 8 * k,
                           smem_desc_sw128(sv + (uint32_t)k * 2048u, 16, 1024), idesc_o, (j | k) != 0);
                mma_commit(&o_done[g]);
            };
            if (ok) ok = mbar_wait(&k_full[0], 0, abort_flag);
            if (ok) {
                tc_fence_after();
                issue_s(0, 0);
                if (has_b) issue_s(1, 0);
            }
            for (int j = 0; j < nkv && ok; ++j) {
                const int s = j % NS;
                if (j + 1 < nkv) {
                    // next S tiles as soon as the softmax warps hold the current ones in registers
                    if (!mbar_wait(&k_full[(j + 1) % NS], ((j + 1) / NS) & 1, abort_flag)) { ok = false; break; }
                    if (!mbar_wait(&s_free[0], j & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    issue_s(0, j + 1);
                    if (has_b) {
                        if (!mbar_wait(&s_free[1], j & 1, abort_flag)) { ok = false; break; }
                        tc_fence_after();
                        issue_s(1, j + 1);
                    }
                }
                if (!mbar_wait(&v_full[s], (j / NS) & 1, abort_flag)) { ok = false; break; }
                if (!mbar_wait(&p_ready[0], j & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                issue_pv(0, j);
                if (has_b) {
                    if (!mbar_wait(&p_ready[1], j & 1, abort_flag)) { ok = false; break; }
                    tc_fence_after();
                    issue_pv(1, j);
                }
                mma_commit(&kv_empty[s]);
            }
        }
    }
    } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    if (warp < 4 || has_b) {
        // ---------------- softmax, O rescaling and output: one query row per thread ----------------
        const int g = warp >> 2;                         // query tile of this warpgroup
        const int q = warp & 3;                          // tensor-memory lane quadrant of this warp
        const int row = q0 + g * BQ + q * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t s_addr = lane_addr + g * BKV, p_addr = lane_addr + kPCol + g * DH,
                       o_addr = lane_addr + kOCol + g * DH;
        const float sl = args.scale_log2;
        float m_l2 = 0.f, l_run = 0.f;                   // running maximum (times scale*log2 e) and sum
        bool ok = true;
        for (int j = 0; j < nkv && ok; ++j) {
            const int valid = min(BKV, N - j * BKV);
            // the warp moves as one through the collective tensor-memory accesses below
            if (!__all_sync(0xffffffffu, mbar_wait(&s_full[g], j & 1, abort_flag))) { ok = false; break; }
            tc_fence_after();
            // All 128 columns are read even on a partial key tile: columns past the keys the MMA
            // wrote hold old values, which the masks below never let through.
            uint32_t r[128];
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_ld_32x32(s_addr + c * 32, r + c * 32);
            tmem_wait_ld();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&s_free[g]);      // the next Q K^T may overwrite S now
            // running maximum: raised only when the tile tops it by more than 2^kRescaleGap
            const float mx_l2 = (valid == BKV ? row_max<false>(r, valid) : row_max<true>(r, valid)) * sl;
            if (j == 0) {
                m_l2 = mx_l2;
            } else if (__any_sync(0xffffffffu, mx_l2 > m_l2 + kRescaleGap)) {
                // rare: rescale O and the sum; O += P V of the previous key tile must have retired
                if (!__all_sync(0xffffffffu, mbar_wait(&o_done[g], (j - 1) & 1, abort_flag))) { ok = false; break; }
                tc_fence_after();
                const bool raise = mx_l2 > m_l2 + kRescaleGap;
                const float alpha = raise ? ex2(m_l2 - mx_l2) : 1.f;
                if (raise) m_l2 = mx_l2;
                l_run *= alpha;
#pragma unroll
                for (int c = 0; c < 2; ++c) {
                    uint32_t o[32];
                    tmem_ld_32x32(o_addr + c * 32, o);
                    tmem_wait_ld();
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                    tmem_st_32x32(o_addr + c * 32, o);
                }
                tmem_wait_st();
            }
            // The two softmax warps of a scheduler (tile A's and tile B's warp q) take turns at
            // the exponent pass: the MUFU unit is the bottleneck, and run one at a time each pass
            // overlaps the other warp's loads, stores and waits instead of its exponentials.
            // Order: A0 B0 A1 B1 ...
            if (kPingPong && has_b && j < kPingPongTiles && (g == 1 || j > 0)) {
                const uint32_t par = (g == 1 ? j : j - 1) & 1;
                if (!__all_sync(0xffffffffu, mbar_wait(&turn[(g ^ 1) * 4 + q], par, abort_flag))) { ok = false; break; }
            }
            const float lsum = valid == BKV ? exp_pass<false>(r, sl, -m_l2, valid) : exp_pass<true>(r, sl, -m_l2, valid);
            if (kPingPong && has_b && lane == 0) mbar_arrive(&turn[g * 4 + q]);
            if (j > 0) {
                // P V of the previous key tile reads the P columns: it must have retired
                if (!__all_sync(0xffffffffu, mbar_wait(&o_done[g], (j - 1) & 1, abort_flag))) { ok = false; break; }
                tc_fence_after();
            }
            l_run += lsum;
#pragma unroll
            for (int c = 0; c < 4; ++c) tmem_st_32x16(p_addr + c * 16, r + c * 16);
            tmem_wait_st();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&p_ready[g]);
        }
        // epilogue: O / l -> bf16 -> global
        if (ok && __all_sync(0xffffffffu, mbar_wait(&o_done[g], (nkv - 1) & 1, abort_flag))) {
            tc_fence_after();
            const float inv = 1.f / l_run;
            __nv_bfloat16* op = args.out + ((size_t)((size_t)b * N + row) * args.H + h) * DH;
            uint32_t o[64];
            tmem_ld_32x32(o_addr, o);
            tmem_ld_32x32(o_addr + 32, o + 32);
            tmem_wait_ld();
            if (row < N) {
#pragma unroll
                for (int g8 = 0; g8 < 8; ++g8) {
                    uint32_t w[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e)
                        w[e] = pack_bf16(__uint_as_float(o[8 * g8 + 2 * e]) * inv, __uint_as_float(o[8 * g8 + 2 * e + 1]) * inv);
                    *reinterpret_cast<uint4*>(op + g8 * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                }
            }
        }
    }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicExch(args.status, RS_DEV_TIMEOUT);
    if (warp == 9) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// [B, N, H, 64] view with element strides; box = 128 rows of one head of one sample.
bool make_tmap_qkv(void* encode_fn, CUtensorMap* out, const void* base, int B, int N, int H, long long bs,
                   long long rs_, long long hs) {
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(encode_fn);
    const cuuint64_t dims[4] = {64, (cuuint64_t)H, (cuuint64_t)N, (cuuint64_t)B};
    // a dimension of extent 1 never uses its stride; give it a harmless valid one
    const cuuint64_t hs_b = (H > 1 ? (cuuint64_t)hs : 64) * 2, rs_b = (N > 1 ? (cuuint64_t)rs_ : 64) * 2,
                     bs_b = (B > 1 ? (cuuint64_t)bs : 64) * 2;
    const cuuint64_t strides[3] = {hs_b, rs_b, bs_b};
    const cuuint32_t box[4] = {64, 1, 128, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

bool attn_tc_supported(const rs_attn_desc& d) {
    if (d.dtype != RS_BF16 || d.head_dim != 64 || d.B > 65535 || d.H > 65535) return false;
    const long long st[9] = {d.q_batch_stride, d.q_row_stride, d.q_head_stride, d.k_batch_stride, d.k_row_stride,
                             d.k_head_stride,  d.v_batch_stride, d.v_row_stride, d.v_head_stride};
    for (int i = 0; i < 9; ++i)
        if (st[i] < 0 || (st[i] % 8) != 0 || st[i] >= (1ll << 38)) return false;
    // a stride of an extent > 1 dimension must be positive
    if ((d.H > 1 && (!d.q_head_stride || !d.k_head_stride || !d.v_head_stride)) ||
        (d.N > 1 && (!d.q_row_stride || !d.k_row_stride || !d.v_row_stride)) ||
        (d.B > 1 && (!d.q_batch_stride || !d.k_batch_stride || !d.v_batch_stride)))
        return false;
    return true;
}

cudaError_t launch_attn_tc(rs_ctx* ctx, const rs_attn_desc& d, const void* q, const void* k, const void* v,
                           void* out, cudaStream_t st) {
    if (!ctx->encode_tiled) return cudaErrorNotSupported;
    static bool attr_done = false;
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    CUtensorMap tmQ, tmK, tmV;
    if (!make_tmap_qkv(ctx->encode_tiled, &tmQ, q, d.B, d.N, d.H, d.q_batch_stride, d.q_row_stride, d.q_head_stride) ||
        !make_tmap_qkv(ctx->encode_tiled, &tmK, k, d.B, d.N, d.H, d.k_batch_stride, d.k_row_stride, d.k_head_stride) ||
        !make_tmap_qkv(ctx->encode_tiled, &tmV, v, d.B, d.N, d.H, d.v_batch_stride, d.v_row_stride, d.v_head_stride))
        return cudaErrorInvalidValue;
    AttnArgs args;
    args.out = (__nv_bfloat16*)out;
    args.N = d.N; args.H = d.H;
    const float scale = d.scale != 0.f ? d.scale : 0.125f;
    args.scale_log2 = scale * 1.4426950408889634f;
    args.status = ctx->d_status;
    const dim3 grid((d.N + 2 * BQ - 1) / (2 * BQ), d.H, d.B);
    attn_tc_kernel<<<grid, kThreads, kSmem, st>>>(tmQ, tmK, tmV, args);
    return cudaGetLastError();
}

}  // namespace rs
