// Fused attention on the tensor cores (Eq. sa) for long sequences: three query tiles per CTA.
//
// Same scheme as rs_attn_tc.cu -- S = Q K^T by tcgen05.mma into tensor memory, a softmax warpgroup
// per query tile with a row per thread, P as the tensor-memory A operand of O += P V, lazy
// rescaling -- with the work cut finer so that a third stream fits: key tiles of 64 instead of 128
// keys, hence per query tile 64 columns of S, 32 of P and 64 of O, 480 of the 512 tensor-memory
// columns for three tiles.  With head dimension 64 the special-function unit (the exponentials)
// bounds the kernel, and what keeps that unit from saturating is the serial chain of each
// softmax warp; three warps per scheduler instead of two fill more of its gaps.
// An item is three consecutive 128-row query tiles of one (sample, head), which share the K/V
// tiles streamed through the TMA ring.
#include <math.h>

#include "rs_internal.h"
#include "rs_attn.cuh"
#include "rs_device.cuh"
#include "rs_once.h"
#include "rs_tc.cuh"

namespace rs {

namespace {

using namespace tc;
using namespace attn;

constexpr int BQ = 128, BKV = 64, DH = 64, NG = 3;
constexpr int Q_BYTES = BQ * DH * 2;            // 16 KB: a [128, 64] bf16 tile
constexpr int KV_BYTES = BKV * DH * 2;          // 8 KB: a [64, 64] bf16 tile
constexpr int NS = 5;                           // K/V ring stages
constexpr int kThreads = 512;                   // warps 0-3 / 4-7 / 8-11: softmax of tile 0 / 1 / 2, warp 12: TMA, warp 13: Q K^T, warp 14: P V
// the fourth warpgroup (TMA, MMA and two idle warps) hands registers to the three softmax warpgroups
constexpr int kLaunchRegs = 128, kSoftmaxRegs = 152, kOtherRegs = 56;
static_assert(384 * kSoftmaxRegs + 128 * kOtherRegs <= kThreads * kLaunchRegs, "register pool of the CTA");
constexpr int kSCol = 0, kPCol = NG * BKV, kOCol = kPCol + NG * (BKV / 2);   // S 0..191, P 192..287, O 288..479
constexpr int kTmemCols = 512;
constexpr float kRescaleGap = 8.f;              // log2 units the tile maximum may exceed the running one
// shared memory: Q[2 buffers][NG] | K[NS] | V[NS] | output staging | barriers
constexpr int OFF_Q = 0, OFF_K = 2 * NG * Q_BYTES, OFF_V = OFF_K + NS * KV_BYTES;
constexpr int OFF_OST = OFF_V + NS * KV_BYTES;  // output staging: 12 softmax warps x 32 rows x 128 bytes
constexpr int OFF_BAR = OFF_OST + 4 * NG * 4096;
constexpr size_t kSmem = (size_t)OFF_BAR + 512 + 1024 /*alignment slack*/;
static_assert(kOCol + NG * DH <= kTmemCols, "tensor-memory columns");
static_assert(kSmem <= 232448, "shared memory of one CTA");

// Items: first the groups of three query tiles of every (sample, head) -- n3 of them, per3 to a head --
// then, where the tile count is not a multiple of three, one item per head with the tail_ng tiles left
// over (n_tail of them).  CTA c takes the groups c, c + G, ... and then tails: tail number
// tail_pos + k * tail_stride for k = 0, 1, ..., where tail_pos = c - tail_first (CTAs before tail_first
// take none, unless the tails wrap around: tail_wrap = 1, position (c - tail_first) mod G).
struct Attn3Args {
    int N, H;
    int per3, n3, n_tail, tail_ng;
    int tail_first, tail_stride, tail_wrap;
    float scale_log2;        // scale * log2(e)
    int* status;
};

struct Item3 {
    int b, h, q0;            // sample, head, first query row of tile 0 (tile g starts at q0 + g * 128)
    int ng;                  // query tiles present: 1 .. 3
};
__device__ __forceinline__ Item3 decode_item3(const Attn3Args& a, int w) {
    Item3 it;
    int bh;
    if (w < a.n3) {
        bh = w / a.per3;
        it.q0 = (w - bh * a.per3) * NG * BQ;
        it.ng = NG;
    } else {
        bh = w - a.n3;
        it.q0 = a.per3 * NG * BQ;
        it.ng = a.tail_ng;
    }
    it.b = bh / a.H;
    it.h = bh - it.b * a.H;
    return it;
}
// The k-th item of this CTA, or -1 when it has none left.
__device__ __forceinline__ int item_of(const Attn3Args& a, int k) {
    const int c = blockIdx.x, G = gridDim.x;
    const int mine3 = c < a.n3 ? (a.n3 - c + G - 1) / G : 0;
    if (k < mine3) return c + k * G;
    int pos = c - a.tail_first;
    if (pos < 0) {
        if (!a.tail_wrap) return -1;
        pos += G;
    }
    const int s = pos + (k - mine3) * a.tail_stride;
    return s < a.n_tail ? a.n3 + s : -1;
}

// Maximum of a 64-column row of S in registers.  MASKED: only the first `valid` columns are keys.
template <bool MASKED>
__device__ __forceinline__ float row_max64(const uint32_t (&r)[BKV], int valid) {
    float m[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) m[c] = -INFINITY;
#pragma unroll
    for (int i = 0; i < BKV; i += 16) {               // eight independent chains: latency, not count, is the cost
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float a = __uint_as_float(r[i + 2 * c]), b = __uint_as_float(r[i + 2 * c + 1]);
            if (MASKED) {
                if (i + 2 * c >= valid) a = -INFINITY;
                if (i + 2 * c + 1 >= valid) b = -INFINITY;
            }
            m[c] = max3(m[c], a, b);
        }
    }
    return max3(max3(m[0], m[1], m[2]), max3(m[3], m[4], m[5]), fmaxf(m[6], m[7]));
}

// p_i = exp2(s_i * sl + mneg) for the first `valid` of the 64 keys (0 for the rest), packed to bf16
// pairs in place (r[0 .. 32) on return); returns the sum of the unrounded p_i.
template <bool MASKED>
__device__ __forceinline__ float exp_pass64(uint32_t (&r)[BKV], float sl, float mneg, int valid) {
    const uint64_t sl2 = pack2(sl, sl), mneg2 = pack2(mneg, mneg);
    uint64_t l01 = pack2(0.f, 0.f), l23 = l01;
#pragma unroll
    for (int i = 0; i < BKV; i += 4) {
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
attn_tc3_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
                const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO, const Attn3Args args) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint64_t* q_full = bars;                 // [2] Q tiles of the item landed in buffer 0 / 1
    uint64_t* q_empty = bars + 2;            // [2] every Q K^T of the item in that buffer retired
    uint64_t* k_full = bars + 4;             // [NS] K tile landed
    uint64_t* v_full = k_full + NS;          // [NS] V tile landed
    uint64_t* k_empty = k_full + 2 * NS;     // [NS] every Q K^T reading the K stage retired
    uint64_t* v_empty = k_full + 3 * NS;     // [NS] every P V reading the V stage retired
    uint64_t* s_full = k_full + 4 * NS;      // [NG] S of the tile complete in tensor memory
    uint64_t* p_ready = s_full + NG;         // [NG] P written (one arrival per softmax warp)
    uint64_t* o_done = s_full + 2 * NG;      // [NG] O += P V retired
    uint64_t* s_free = s_full + 3 * NG;      // [NG] S row in registers, columns reusable (one arrival per warp)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_full + 4 * NG);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmO);
        for (int i = 0; i < 2; ++i) { mbar_init(&q_full[i], 1); mbar_init(&q_empty[i], 1); }
        for (int s = 0; s < NS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&v_full[s], 1); mbar_init(&k_empty[s], 1); mbar_init(&v_empty[s], 1); }
        for (int g = 0; g < NG; ++g) { mbar_init(&s_full[g], 1); mbar_init(&p_ready[g], 4); mbar_init(&o_done[g], 1); mbar_init(&s_free[g], 4); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 13) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    // Everything above touched no global memory and may overlap the previous kernel's tail.
    grid_dep_launch();
    grid_dep_wait();
    const int nkv = (args.N + BKV - 1) / BKV;           // key tiles per query tile

    if (warp >= 12) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
    if (warp == 12) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            uint32_t kv_it = 0, item_n = 0;
            bool ok = true;
            for (int w = item_of(args, 0); w >= 0 && ok; w = item_of(args, ++item_n)) {
                const Item3 it = decode_item3(args, w);
                const uint32_t qb = item_n & 1u;
                if (!mbar_wait(&q_empty[qb], ((item_n >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                mbar_expect_tx(&q_full[qb], it.ng * Q_BYTES);
                for (int g = 0; g < it.ng; ++g)
                    tma_load_4d(smem + OFF_Q + (qb * NG + g) * Q_BYTES, &tmQ, &q_full[qb], 0, it.h, it.q0 + g * BQ, it.b);
                for (int t = 0; t < nkv; ++t, ++kv_it) {
                    const int s = kv_it % NS;
                    if (!mbar_wait(&k_empty[s], ((kv_it / NS) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(&k_full[s], KV_BYTES);
                    tma_load_4d(smem + OFF_K + s * KV_BYTES, &tmK, &k_full[s], 0, it.h, t * BKV, it.b);
                    if (!mbar_wait(&v_empty[s], ((kv_it / NS) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    mbar_expect_tx(&v_full[s], KV_BYTES);
                    tma_load_4d(smem + OFF_V + s * KV_BYTES, &tmV, &v_full[s], 0, it.h, t * BKV, it.b);
                }
            }
            // every copy started here must have landed before the CTA exits
            for (uint32_t n = item_n > 2 ? item_n - 2 : 0; n < item_n && ok; ++n)
                ok = mbar_wait(&q_full[n & 1u], (n >> 1) & 1u, abort_flag);
            for (uint32_t t = kv_it > NS ? kv_it - NS : 0; t < kv_it && ok; ++t)
                ok = mbar_wait(&k_full[t % NS], (t / NS) & 1u, abort_flag) && mbar_wait(&v_full[t % NS], (t / NS) & 1u, abort_flag);
        }
    } else if (warp == 13) {
        // ---------------- Q K^T issuer: S_g = Q_g K^T, both operands K-major ----------------
        // It runs ahead of the softmax warps as far as the S columns allow: the S of a tile may be
        // overwritten once that tile's softmax warps have its row in registers.
        if (elect_one()) {
            constexpr uint32_t idesc_s_full = idesc_bf16(BQ, BKV, 0, 0);
            constexpr uint32_t kQ16 = Q_BYTES >> 4, kKV16 = KV_BYTES >> 4;
            const uint32_t desc_hi = smem_desc_hi(smem_desc_sw128(0, 16, 1024));
            const uint32_t q_lo = smem_desc_lo(smem_desc_sw128(smem_u32(smem + OFF_Q), 16, 1024));
            const uint32_t k_lo = smem_desc_lo(smem_desc_sw128(smem_u32(smem + OFF_K), 16, 1024));
            uint32_t ns[NG] = {0, 0, 0};                 // S tiles issued so far per query tile
            uint32_t item_n = 0, t = 0;
            bool ok = true;
            for (int w = item_of(args, 0); w >= 0 && ok; w = item_of(args, ++item_n)) {
                const int ng = decode_item3(args, w).ng;
                const uint32_t qb = item_n & 1u;
                if (!mbar_wait(&q_full[qb], (item_n >> 1) & 1u, abort_flag)) { ok = false; break; }
                for (int j = 0; j < nkv && ok; ++j, ++t) {
                    const int stage = t % NS, valid = min(BKV, args.N - j * BKV);
                    if (!mbar_wait(&k_full[stage], (t / NS) & 1u, abort_flag)) { ok = false; break; }
                    const uint32_t idesc_s = valid == BKV ? idesc_s_full : idesc_bf16(BQ, (valid + 15) & ~15, 0, 0);
                    const uint32_t dk = k_lo + (uint32_t)stage * kKV16;
#pragma unroll
                    for (int g = 0; g < NG; ++g) {
                        if (g >= ng || !ok) continue;
                        if (ns[g] > 0 && !mbar_wait(&s_free[g], (ns[g] - 1) & 1u, abort_flag)) { ok = false; continue; }
                        tc_fence_after();
                        const uint32_t dq = q_lo + (qb * NG + g) * kQ16;
#pragma unroll
                        for (int k = 0; k < DH / 16; ++k)    // 16 head-dimension columns = 32 bytes per step
                            mma_ss_lh(tmem_base + kSCol + g * BKV, dq + 2u * k, dk + 2u * k, desc_hi, idesc_s, k != 0);
                        mma_commit(&s_full[g]);
                        ++ns[g];
                    }
                    if (ok) mma_commit(&k_empty[stage]);
                }
                if (ok) mma_commit(&q_empty[qb]);
            }
        }
    } else if (warp == 14) {
        // ---------------- P V issuer: O_g (+)= P_g V ----------------
        // P from tensor memory (bf16 pairs, 8 columns per 16 keys), V MN-major (head dimension
        // contiguous), 16 keys = 2048 bytes per slab.
        if (elect_one()) {
            constexpr uint32_t idesc_o = idesc_bf16(BQ, DH, 0, 1);
            constexpr uint32_t kKV16 = KV_BYTES >> 4;
            const uint32_t desc_hi = smem_desc_hi(smem_desc_sw128(0, 16, 1024));
            const uint32_t v_lo = smem_desc_lo(smem_desc_sw128(smem_u32(smem + OFF_V), 16, 1024));
            uint32_t np[NG] = {0, 0, 0};                 // P V products issued so far per query tile
            uint32_t t = 0, item_n = 0;
            bool ok = true;
            for (int w = item_of(args, 0); w >= 0 && ok; w = item_of(args, ++item_n)) {
                const int ng = decode_item3(args, w).ng;
                for (int j = 0; j < nkv && ok; ++j, ++t) {
                    const int stage = t % NS, valid = min(BKV, args.N - j * BKV);
                    if (!mbar_wait(&v_full[stage], (t / NS) & 1u, abort_flag)) { ok = false; break; }
                    const uint32_t dv = v_lo + (uint32_t)stage * kKV16;
                    const int ksteps = (valid + 15) >> 4;
#pragma unroll
                    for (int g = 0; g < NG; ++g) {
                        if (g >= ng || !ok) continue;
                        if (!mbar_wait(&p_ready[g], np[g] & 1u, abort_flag)) { ok = false; continue; }
                        tc_fence_after();
                        const uint32_t o_col = tmem_base + kOCol + g * DH, p_col = tmem_base + kPCol + g * (BKV / 2);
                        for (int k = 0; k < ksteps; ++k)
                            mma_ts_lh(o_col, p_col + 8 * k, dv + 128u * k, desc_hi, idesc_o, !(j == 0 && k == 0));
                        mma_commit(&o_done[g]);
                        ++np[g];
                    }
                    if (ok) mma_commit(&v_empty[stage]);
                }
            }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
        // ---------------- softmax, O rescaling and output: one query row per thread ----------------
        const int g = warp >> 2;                         // query tile of this warpgroup
        const int q = warp & 3;                          // tensor-memory lane quadrant of this warp
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t s_addr = lane_addr + kSCol + g * BKV, p_addr = lane_addr + kPCol + g * (BKV / 2),
                       o_addr = lane_addr + kOCol + g * DH;
        const float sl = args.scale_log2;
        uint32_t cnt = 0;                                // key tiles this warpgroup has walked through
        bool ok = true;
        uint32_t item_n = 0;
        for (int w = item_of(args, 0); w >= 0 && ok; w = item_of(args, ++item_n)) {
            const Item3 it = decode_item3(args, w);
            if (g >= it.ng) continue;
            float m_l2 = 0.f, l_run = 0.f;               // running maximum (times scale*log2 e) and sum
            for (int j = 0; j < nkv && ok; ++j, ++cnt) {
                const int valid = min(BKV, args.N - j * BKV);
                // the warp moves as one through the collective tensor-memory accesses below
                if (!__all_sync(0xffffffffu, mbar_wait(&s_full[g], cnt & 1u, abort_flag))) { ok = false; break; }
                tc_fence_after();
                // All 64 columns are read even on a partial key tile: columns past the keys the MMA
                // wrote hold old values, which the masks never let through.
                uint32_t r[BKV];
                tmem_ld_32x32(s_addr, r);
                tmem_ld_32x32(s_addr + 32, r + 32);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_free[g]);  // the next Q K^T may overwrite S now
                // running maximum: raised only when the tile tops it by more than 2^kRescaleGap
                const float mx = valid == BKV ? row_max64<false>(r, valid) : row_max64<true>(r, valid);
                const float mx_l2 = mx * sl;
                if (j == 0) {
                    m_l2 = mx_l2;
                } else if (__any_sync(0xffffffffu, mx_l2 > m_l2 + kRescaleGap)) {
                    // rare: rescale O and the sum; O += P V of the previous key tile must have retired
                    if (!__all_sync(0xffffffffu, mbar_wait(&o_done[g], (cnt - 1) & 1u, abort_flag))) { ok = false; break; }
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
                l_run += valid == BKV ? exp_pass64<false>(r, sl, -m_l2, valid) : exp_pass64<true>(r, sl, -m_l2, valid);
                if (cnt > 0) {
                    // P V of the previous key tile reads the P columns: it must have retired
                    if (!__all_sync(0xffffffffu, mbar_wait(&o_done[g], (cnt - 1) & 1u, abort_flag))) { ok = false; break; }
                    tc_fence_after();
                }
                tmem_st_32x32(p_addr, r);
                tmem_wait_st();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&p_ready[g]);
            }
            // epilogue of the item: O / l -> bf16 -> global
            if (!ok || !__all_sync(0xffffffffu, mbar_wait(&o_done[g], (cnt - 1) & 1u, abort_flag))) { ok = false; break; }
            tc_fence_after();
            const float inv = 1.f / l_run;
            uint32_t o[64];
            tmem_ld_32x32(o_addr, o);
            tmem_ld_32x32(o_addr + 32, o + 32);
            tmem_wait_ld();
            // The warp's 32 rows x 64 values go to its own slab of shared memory (128-byte rows,
            // 16-byte pieces XOR-swizzled like the tensor map's box) and leave with one TMA store,
            // which drops the rows past N.
            if (lane == 0) tma_store_wait_read<0>();     // the slab's previous store has read it
            __syncwarp();
            uint8_t* slab = smem + OFF_OST + (g * 4 + q) * 4096 + (lane >> 3) * 1024 + (lane & 7) * 128;
#pragma unroll
            for (int g8 = 0; g8 < 8; ++g8) {
                uint32_t wv[4];
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    wv[e] = pack_bf16(__uint_as_float(o[8 * g8 + 2 * e]) * inv, __uint_as_float(o[8 * g8 + 2 * e + 1]) * inv);
                *reinterpret_cast<uint4*>(slab + ((g8 ^ (lane & 7)) << 4)) = make_uint4(wv[0], wv[1], wv[2], wv[3]);
            }
            fence_async_smem();
            __syncwarp();
            const int row0 = it.q0 + g * BQ + q * 32;
            if (lane == 0 && row0 < args.N) {
                tma_store_4d(&tmO, smem + OFF_OST + (g * 4 + q) * 4096, 0, it.h, row0, it.b);
                tma_store_commit();
            }
        }
        if (lane == 0) tma_store_wait<0>();              // every output row written before the CTA exits
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicExch(args.status, RS_DEV_TIMEOUT);
    if (warp == 13) {
        __syncwarp();
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

}  // namespace

// Where the leftover-tile items go, and the load of the longest CTA under it, in tenths of a group
// of three tiles (a group or two leftover tiles 10, one leftover tile 7: measured).  wrap = 0: the CTAs
// that the last, incomplete round of groups left out take the tails, up to two each; wrap = 1: the
// tails continue the round robin over all CTAs.
static long long tc3_load(long long BH, int N, int G, int wrap) {
    const int tiles = (N + BQ - 1) / BQ, per3 = tiles / NG, tail_ng = tiles - per3 * NG;
    const long long n3 = BH * per3, n_tail = tail_ng ? BH : 0;
    const int r = (int)(n3 % G), idle = G - r;
    if (!wrap && n_tail > 2ll * idle) return -1;
    const int stride = wrap ? G : idle, tail_cost = tail_ng == 1 ? 7 : 10;
    long long worst = 0;
    for (int c = 0; c < G; ++c) {
        long long load = c < n3 ? 10 * ((n3 - c + G - 1) / G) : 0;
        int pos = c - r;
        if (pos < 0) {
            if (!wrap) { worst = load > worst ? load : worst; continue; }
            pos += G;
        }
        if (pos < n_tail) load += tail_cost * ((n_tail - pos + stride - 1) / stride);
        worst = load > worst ? load : worst;
    }
    return worst;
}
long long attn_tc3_plan(long long BH, int N, int G, int* wrap) {
    const long long a = tc3_load(BH, N, G, 0), b = tc3_load(BH, N, G, 1);
    *wrap = (a < 0 || b < a) ? 1 : 0;
    return *wrap ? b : a;
}

// tmK, tmV: boxes of 64 rows; tmQ: 128 rows; tmO: 32 rows.
cudaError_t launch_attn_tc3(rs_ctx* ctx, const rs_attn_desc& d, const CUtensorMap& tmQ, const CUtensorMap& tmK,
                            const CUtensorMap& tmV, const CUtensorMap& tmO, int wrap, cudaStream_t st) {
    if (d.N <= BQ) return cudaErrorInvalidValue;          // one query tile: the two-heads-per-item kernel's
    static PerDeviceOnce attr_once;   // the attribute belongs to the device current at the call
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = (cudaError_t)attr_once.run(dev, [] {
        return (int)cudaFuncSetAttribute(attn_tc3_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
    });
    if (e != cudaSuccess) return e;
    Attn3Args args;
    args.N = d.N; args.H = d.H;
    const int tiles = (d.N + BQ - 1) / BQ, G = ctx->sm_count;
    const long long BH = (long long)d.B * d.H;
    args.per3 = tiles / NG;
    args.tail_ng = tiles - args.per3 * NG;
    if (BH * (args.per3 + 1) >= (1ll << 30)) return cudaErrorInvalidValue;
    args.n3 = (int)(BH * args.per3);
    args.n_tail = args.tail_ng ? (int)BH : 0;
    const int r = args.n3 % G, idle = G - r;
    if (!wrap && args.n_tail > 2ll * idle) wrap = 1;
    args.tail_first = r;
    args.tail_stride = wrap ? G : idle;
    args.tail_wrap = wrap;
    const float scale = d.scale != 0.f ? d.scale : 0.125f;
    args.scale_log2 = scale * 1.4426950408889634f;
    args.status = ctx->d_status;
    const long long all = (long long)args.n3 + args.n_tail;
    const int grid = all < G ? (int)all : G;
    return launch_pdl(attn_tc3_kernel, dim3(grid), dim3(kThreads), kSmem, st, tmQ, tmK, tmV, tmO, args);
}

}  // namespace rs
