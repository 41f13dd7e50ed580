// Fused attention on the tensor cores (Eq. sa): out = Softmax(Q K^T * scale) V per
// (sample, head), head dimension 64, without ever writing the N x N matrix.
//
// Persistent kernel, one CTA per SM, looping over work items.  An item is two 128-row query
// tiles A and B: for N > 128 two consecutive query tiles of one (sample, head), which share
// the key/value tiles streamed through a TMA ring; for N <= 128 the single query tile of two
// neighbouring heads, each with its own key/value tile.  For each query tile and key tile:
// S = Q K^T (tcgen05.mma, fp32 in tensor memory)  ->  a softmax warpgroup (a row per thread)
// pulls the S row into registers and at once hands the S columns back, so the next Q K^T is
// computed while this tile's exponentials run; it keeps a running maximum and sum and writes
// P = exp2(S*c - m*c) as bf16 into P's own tensor-memory columns  ->  O += P V (tcgen05.mma
// with P as the tensor-memory A operand and the V tile as an MN-major shared-memory B
// operand).  The running maximum is raised only when a tile tops it by more than 2^8 (the
// final division by the row sum gives the exact softmax either way), so O is rarely rescaled
// and the softmax warps do that themselves.  The TMA producer, the MMA issuer and the softmax
// warps each walk the same item list and keep their own phase counters, so loads, Q K^T of the
// next item and the epilogue of the previous one overlap across item boundaries.
#include <math.h>

#include <map>
#include <mutex>
#include <tuple>

#include "rs_internal.h"
#include "rs_attn.cuh"
#include "rs_device.cuh"
#include "rs_once.h"
#include "rs_tc.cuh"

namespace rs {

namespace {

using namespace tc;
using namespace attn;

constexpr int BQ = 128, BKV = 128, DH = 64;
constexpr int TILE_BYTES = 128 * DH * 2;        // 16 KB: a [128, 64] bf16 tile
constexpr int NS = 4;                           // K/V ring stages
constexpr int kThreads = 384;                   // warps 0-3 / 4-7: softmax of tile A / B, warp 8: TMA, warp 9: MMA
constexpr int kSoftmaxRegs = 216, kOtherRegs = 72;   // per-thread register budgets after the warpgroups re-split the pool
constexpr int kTmemCols = 512;                  // S_A 0..127, S_B 128..255, P_A 256..319, P_B 320..383, O_A 384..447, O_B 448..511
constexpr int kPCol = 256, kOCol = 384;
constexpr float kRescaleGap = 8.f;              // log2 units the tile maximum may exceed the running one
// shared memory: Q[2 buffers][A, B] | K[NS] | V[NS] | output staging | barriers
constexpr int OFF_Q = 0, OFF_K = 4 * TILE_BYTES, OFF_V = (4 + NS) * TILE_BYTES;
constexpr int OFF_OST = (4 + 2 * NS) * TILE_BYTES;   // output staging: 8 softmax warps x 32 rows x 128 bytes
constexpr int OFF_BAR = OFF_OST + 8 * 4096;
constexpr size_t kSmem = (size_t)OFF_BAR + 256 + 1024 /*alignment slack*/;

struct AttnArgs {
    __nv_bfloat16* out;      // [B, N, H*64]
    int N, H;
    int dual;                // 1: N <= 128, an item is two heads; 0: an item is two query tiles of one head
    int per;                 // items per (sample, head) [dual = 0] or per sample [dual = 1]
    int n_items;
    // dual = 0: the first n_pair_items items are pairs of query tiles; the rest are single query tiles,
    // tile_count of them for each (sample, head) from first_single_bh on (see launch_attn_tc)
    int n_pair_items, first_single_bh, tile_count;
    float scale_log2;        // scale * log2(e)
    const int* lens;         // optional [B]: sample b attends over its first lens[b] tokens only (clamped to 1 .. N)
    int* status;
};

// One work item, decoded the same way by every role.
struct Item {
    int b, h[2], q0[2];      // sample; head and first query row of tile A / B
    int n;                   // tokens of the sample (N, or its own length)
    int ng;                  // query tiles present: 1 or 2 (0: the item lies past the sample's own length and is skipped)
    int nkv;                 // key tiles per query tile
    int slots;               // K/V ring stages the item consumes
};
__device__ __forceinline__ Item decode_item(const AttnArgs& a, int w) {
    Item it;
    if (a.dual) {
        const int hp = w % a.per;
        it.b = w / a.per;
        it.h[0] = 2 * hp; it.h[1] = 2 * hp + 1;
        it.q0[0] = it.q0[1] = 0;
        it.n = a.lens ? min(max(__ldg(a.lens + it.b), 1), a.N) : a.N;
        it.ng = it.h[1] < a.H ? 2 : 1;
        it.nkv = 1;
        it.slots = it.ng;
    } else {
        int bh;
        if (w < a.n_pair_items) {
            const int qp = w % a.per;
            bh = w / a.per;
            it.q0[0] = qp * 2 * BQ; it.q0[1] = it.q0[0] + BQ;
        } else {
            const int k = w - a.n_pair_items;
            bh = a.first_single_bh + k / a.tile_count;
            it.q0[0] = (k % a.tile_count) * BQ; it.q0[1] = a.N;       // one query tile only
        }
        it.b = bh / a.H;
        it.h[0] = it.h[1] = bh % a.H;
        it.n = a.lens ? min(max(__ldg(a.lens + it.b), 1), a.N) : a.N;
        it.ng = (it.q0[0] < it.n ? 1 : 0) + (it.q0[1] < it.n ? 1 : 0);
        it.nkv = (it.n + BKV - 1) / BKV;
        it.slots = it.nkv;
    }
    return it;
}
// First item at or after w (in this CTA's stride) that has work; n_items if none.
__device__ __forceinline__ int next_item(const AttnArgs& a, int w, int stride) {
    if (!a.lens) return w;
    while (w < a.n_items && decode_item(a, w).ng == 0) w += stride;
    return w;
}

// Maximum of the first NC values of a row of S held in registers.  MASK 0: all NC are keys.
// MASK 1: NC = the 32-column groups that hold keys, so only the last group can hold columns past
// `valid` and only there the elements are tested.  MASK 2: every element is tested.
template <int NC, int MASK>
__device__ __forceinline__ float row_max(const uint32_t (&r)[128], int valid) {
    float m[8];
#pragma unroll
    for (int c = 0; c < 8; ++c) m[c] = -INFINITY;
#pragma unroll
    for (int i = 0; i < NC; i += 16) {               // eight independent chains: latency, not count, is the cost
#pragma unroll
        for (int c = 0; c < 8; ++c) {
            float a = __uint_as_float(r[i + 2 * c]), b = __uint_as_float(r[i + 2 * c + 1]);
            if (MASK == 2 || (MASK == 1 && i >= NC - 32)) {
                if (i + 2 * c >= valid) a = -INFINITY;
                if (i + 2 * c + 1 >= valid) b = -INFINITY;
            }
            m[c] = max3(m[c], a, b);
        }
    }
    return max3(max3(m[0], m[1], m[2]), max3(m[3], m[4], m[5]), fmaxf(m[6], m[7]));
}

// p_i = exp2(s_i * sl + mneg) for the first `valid` of NC keys (0 for the rest; MASK as above),
// packed to bf16 pairs in place (r[0 .. NC/2) on return); returns the sum of the unrounded p_i.
template <int NC, int MASK>
__device__ __forceinline__ float exp_pass(uint32_t (&r)[128], float sl, float mneg, int valid) {
    const uint64_t sl2 = pack2(sl, sl), mneg2 = pack2(mneg, mneg);
    uint64_t l01 = pack2(0.f, 0.f), l23 = l01;
#pragma unroll
    for (int i = 0; i < NC; i += 4) {
        float x0, x1, x2, x3;
        unpack2(ffma2(pack2(__uint_as_float(r[i]), __uint_as_float(r[i + 1])), sl2, mneg2), x0, x1);
        unpack2(ffma2(pack2(__uint_as_float(r[i + 2]), __uint_as_float(r[i + 3])), sl2, mneg2), x2, x3);
        if (MASK == 2 || (MASK == 1 && i >= NC - 32)) {
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

// FINE: partial key tiles are handled by 32-column groups (worth it when a sequence is a few
// tiles long).  Without it the one partial tile of a long sequence is a full tile with every
// element tested, and the kernel carries less code around its inner loop, which that loop feels.
template <bool FINE>
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const __grid_constant__ CUtensorMap tmO, const AttnArgs args) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint64_t* q_full = bars;                 // [2] Q tiles of the item landed in buffer 0 / 1
    uint64_t* q_empty = bars + 2;            // [2] every Q K^T of the item in that buffer retired
    uint64_t* k_full = bars + 4;             // [NS] K tile landed
    uint64_t* v_full = k_full + NS;          // [NS] V tile landed
    uint64_t* kv_empty = k_full + 2 * NS;    // [NS] every MMA reading the stage retired
    uint64_t* s_full = k_full + 3 * NS;      // [2] S of tile A / B complete in tensor memory
    uint64_t* p_ready = s_full + 2;          // [2] P written (one arrival per softmax warp)
    uint64_t* o_done = s_full + 4;           // [2] O += P V retired
    uint64_t* s_free = s_full + 6;           // [2] S row in registers, columns reusable (one arrival per warp)
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(s_full + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV); prefetch_tmap(&tmO);
        for (int i = 0; i < 2; ++i) { mbar_init(&q_full[i], 1); mbar_init(&q_empty[i], 1); }
        for (int s = 0; s < NS; ++s) { mbar_init(&k_full[s], 1); mbar_init(&v_full[s], 1); mbar_init(&kv_empty[s], 1); }
        for (int g = 0; g < 2; ++g) { mbar_init(&s_full[g], 1); mbar_init(&p_ready[g], 4); mbar_init(&o_done[g], 1); mbar_init(&s_free[g], 4); }
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
    // Everything above touched no global memory and may overlap the previous kernel's tail.
    grid_dep_launch();
    grid_dep_wait();
    // The third warpgroup (TMA, MMA and two idle warps) hands most of its registers to the
    // two softmax warpgroups, which hold a whole 128-column row of S per thread.
    if (warp >= 8) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kOtherRegs));
    if (warp == 8) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            uint32_t kv_it = 0, item_n = 0;
            bool ok = true;
            for (int w = next_item(args, blockIdx.x, gridDim.x); w < args.n_items && ok; w = next_item(args, w + gridDim.x, gridDim.x), ++item_n) {
                const Item it = decode_item(args, w);
                const uint32_t qb = item_n & 1u;
                if (!mbar_wait(&q_empty[qb], ((item_n >> 1) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                mbar_expect_tx(&q_full[qb], it.ng * TILE_BYTES);
#pragma unroll
                for (int g = 0; g < 2; ++g)
                    if (g < it.ng) tma_load_4d(smem + OFF_Q + (qb * 2 + g) * TILE_BYTES, &tmQ, &q_full[qb], 0, it.h[g], it.q0[g], it.b);
                for (int t = 0; t < it.slots; ++t, ++kv_it) {
                    const int s = kv_it % NS;
                    if (!mbar_wait(&kv_empty[s], ((kv_it / NS) & 1u) ^ 1u, abort_flag)) { ok = false; break; }
                    const int head = (args.dual && t == 1) ? it.h[1] : it.h[0], row0 = args.dual ? 0 : t * BKV;
                    mbar_expect_tx(&k_full[s], TILE_BYTES);
                    tma_load_4d(smem + OFF_K + s * TILE_BYTES, &tmK, &k_full[s], 0, head, row0, it.b);
                    mbar_expect_tx(&v_full[s], TILE_BYTES);
                    tma_load_4d(smem + OFF_V + s * TILE_BYTES, &tmV, &v_full[s], 0, head, row0, it.b);
                }
            }
            // every copy started here must have landed before the CTA exits
            for (uint32_t n = item_n > 2 ? item_n - 2 : 0; n < item_n && ok; ++n)
                ok = mbar_wait(&q_full[n & 1u], (n >> 1) & 1u, abort_flag);
            for (uint32_t t = kv_it > NS ? kv_it - NS : 0; t < kv_it && ok; ++t)
                ok = mbar_wait(&k_full[t % NS], (t / NS) & 1u, abort_flag) && mbar_wait(&v_full[t % NS], (t / NS) & 1u, abort_flag);
        }
    } else if (warp == 9) {
        // ---------------- MMA issuer ----------------
        if (elect_one() && next_item(args, blockIdx.x, gridDim.x) < args.n_items) {
            constexpr uint32_t idesc_o = idesc_bf16(BQ, DH, 0, 1), idesc_s_full = idesc_bf16(BQ, BKV, 0, 0);
            // descriptors as halves: per product only the low half moves (address >> 4)
            constexpr uint32_t kTile16 = TILE_BYTES >> 4;
            const uint32_t desc_hi = smem_desc_hi(smem_desc_sw128(0, 16, 1024));
            const uint32_t q_lo = smem_desc_lo(smem_desc_sw128(smem_u32(smem + OFF_Q), 16, 1024));
            const uint32_t k_lo = smem_desc_lo(smem_desc_sw128(smem_u32(smem + OFF_K), 16, 1024));
            const uint32_t v_lo = smem_desc_lo(smem_desc_sw128(smem_u32(smem + OFF_V), 16, 1024));
            uint32_t ns[2] = {0, 0}, np[2] = {0, 0};     // S tiles / P V products issued so far per query tile
            bool ok = true;
            // S_g = Q_g K^T : both operands K-major (head dimension contiguous).  The S columns must
            // have been read by the softmax warps of the previous tile first.
            auto issue_s = [&](int g, uint32_t qb, int stage, int valid) {
                if (ns[g] > 0 && !mbar_wait(&s_free[g], (ns[g] - 1) & 1u, abort_flag)) { ok = false; return; }
                tc_fence_after();
                const uint32_t idesc_s = valid == BKV ? idesc_s_full : idesc_bf16(BQ, (valid + 15) & ~15, 0, 0);
                const uint32_t dq = q_lo + (qb * 2 + g) * kTile16, dk = k_lo + (uint32_t)stage * kTile16;
#pragma unroll
                for (int k = 0; k < DH / 16; ++k)        // 16 head-dimension columns = 32 bytes per step
                    mma_ss_lh(tmem_base + g * BKV, dq + 2u * k, dk + 2u * k, desc_hi, idesc_s, k != 0);
                mma_commit(&s_full[g]);
                ++ns[g];
            };
            // O_g (+)= P_g V : P from tensor memory (bf16 pairs, 8 columns per 16 keys), V MN-major
            // (head dimension contiguous), 16 keys = 2048 bytes per slab.
            auto issue_pv = [&](int g, int stage, int valid, bool first) {
                if (!mbar_wait(&p_ready[g], np[g] & 1u, abort_flag)) { ok = false; return; }
                tc_fence_after();
                const uint32_t dv = v_lo + (uint32_t)stage * kTile16;
                const uint32_t o_col = tmem_base + kOCol + g * DH, p_col = tmem_base + kPCol + g * DH;
                if (valid == BKV) {
#pragma unroll
                    for (int k = 0; k < BKV / 16; ++k)
                        mma_ts_lh(o_col, p_col + 8 * k, dv + 128u * k, desc_hi, idesc_o, k == 0 ? !first : 1u);
                } else {
                    const int ksteps = (valid + 15) >> 4;
                    for (int k = 0; k < ksteps; ++k)
                        mma_ts_lh(o_col, p_col + 8 * k, dv + 128u * k, desc_hi, idesc_o, !(first && k == 0));
                }
                mma_commit(&o_done[g]);
                ++np[g];
            };
            // Issues the Q K^T of step j of query tile g of an item; kv0 = ring position of the item's
            // first K/V slot.
            auto issue_s_one = [&](const Item& it, uint32_t qb, uint32_t kv0, int j, int g) {
                const uint32_t t = kv0 + (args.dual ? g : j);
                if (!mbar_wait(&k_full[t % NS], (t / NS) & 1u, abort_flag)) { ok = false; return; }
                issue_s(g, qb, t % NS, min(BKV, it.n - j * BKV));
            };

            uint32_t item_n = 0, kv0 = 0;
            int w = next_item(args, blockIdx.x, gridDim.x);
            Item cur = decode_item(args, w);
            ok = mbar_wait(&q_full[0], 0, abort_flag);
#pragma unroll
            for (int g = 0; g < 2; ++g)
                if (ok && g < cur.ng) issue_s_one(cur, 0, kv0, 0, g);
            while (ok) {
                const uint32_t qb = item_n & 1u;
                const int wn = next_item(args, w + gridDim.x, gridDim.x);
                Item nxt = cur;
                for (int j = 0; j < cur.nkv && ok; ++j) {
                    // Look ahead, per query tile: the tile's next Q K^T (of this item, or the first of the
                    // next item) goes to the tensor pipe before its P V of this step, which still waits
                    // for the exponentials.  Tile by tile, not step by step: tile A's last P V of an item
                    // then does not queue behind a Q K^T that waits for tile B, which runs half a pass later.
                    const bool last = j + 1 == cur.nkv;
                    const bool ahead = !last || wn < args.n_items;
                    const uint32_t nb = last ? (item_n + 1) & 1u : qb;
                    if (last && ahead) {
                        nxt = decode_item(args, wn);
                        if (!mbar_wait(&q_full[nb], ((item_n + 1) >> 1) & 1u, abort_flag)) { ok = false; break; }
                    }
                    const Item& sit = last ? nxt : cur;
                    const uint32_t skv0 = last ? kv0 + cur.slots : kv0;
                    const int sj = last ? 0 : j + 1;
                    const int valid = min(BKV, cur.n - j * BKV);
#pragma unroll
                    for (int g = 0; g < 2; ++g) {
                        if (!ok) break;
                        if (ahead && g < sit.ng) issue_s_one(sit, nb, skv0, sj, g);
                        if (!ok || g >= cur.ng) continue;
                        const uint32_t t = kv0 + (args.dual ? g : j);
                        if (!mbar_wait(&v_full[t % NS], (t / NS) & 1u, abort_flag)) { ok = false; break; }
                        issue_pv(g, t % NS, valid, j == 0);
                        if (ok && (args.dual || g == cur.ng - 1)) mma_commit(&kv_empty[t % NS]);   // stage done
                    }
                }
                if (!ok) break;
                mma_commit(&q_empty[qb]);
                kv0 += cur.slots;
                ++item_n;
                w = wn;
                if (w >= args.n_items) break;
                cur = nxt;
            }
        }
    }
    } else {
    asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kSoftmaxRegs));
    {
        // ---------------- softmax, O rescaling and output: one query row per thread ----------------
        const int g = warp >> 2;                         // query tile of this warpgroup
        const int q = warp & 3;                          // tensor-memory lane quadrant of this warp
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const uint32_t s_addr = lane_addr + g * BKV, p_addr = lane_addr + kPCol + g * DH,
                       o_addr = lane_addr + kOCol + g * DH;
        const float sl = args.scale_log2;
        uint32_t cnt = 0, item_n = 0;                    // tiles / items this warpgroup has walked through
        bool ok = true;
        for (int w = blockIdx.x; w < args.n_items && ok; w += gridDim.x, ++item_n) {
            const Item it = decode_item(args, w);
            if (g >= it.ng) continue;
            float m_l2 = 0.f, l_run = 0.f;               // running maximum (times scale*log2 e) and sum
            for (int j = 0; j < it.nkv && ok; ++j, ++cnt) {
                const int valid = min(BKV, it.n - j * BKV);
                // the warp moves as one through the collective tensor-memory accesses below
                if (!__all_sync(0xffffffffu, mbar_wait(&s_full[g], cnt & 1u, abort_flag))) { ok = false; break; }
                tc_fence_after();
                // Whole 32-column groups are read even on a partial key tile: columns past the keys
                // the MMA wrote hold old values, which the masks of the last group never let through.
                uint32_t r[128];
                // columns worth touching: whole 32-column groups, or (lean code) half a tile or all of it
                const int ncol = FINE ? (valid + 31) & ~31 : valid <= 64 ? 64 : BKV;
                tmem_ld_32x32(s_addr, r);
                if (ncol > 32) tmem_ld_32x32(s_addr + 32, r + 32);
                if (ncol > 64) tmem_ld_32x32(s_addr + 64, r + 64);
                if (ncol > 96) tmem_ld_32x32(s_addr + 96, r + 96);
                tmem_wait_ld();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(&s_free[g]);  // the next Q K^T may overwrite S now
                // running maximum: raised only when the tile tops it by more than 2^kRescaleGap
                float mx;
                if (valid == BKV) mx = row_max<128, 0>(r, valid);
                else if (!FINE) mx = ncol == 64 ? row_max<64, 2>(r, valid) : row_max<128, 2>(r, valid);
                else mx = ncol == 128 ? row_max<128, 1>(r, valid) : ncol == 96 ? row_max<96, 1>(r, valid)
                          : ncol == 64 ? row_max<64, 1>(r, valid) : row_max<32, 1>(r, valid);
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
                if (valid == BKV) l_run += exp_pass<128, 0>(r, sl, -m_l2, valid);
                else if (!FINE) l_run += ncol == 64 ? exp_pass<64, 2>(r, sl, -m_l2, valid) : exp_pass<128, 2>(r, sl, -m_l2, valid);
                else l_run += ncol == 128 ? exp_pass<128, 1>(r, sl, -m_l2, valid) : ncol == 96 ? exp_pass<96, 1>(r, sl, -m_l2, valid)
                              : ncol == 64 ? exp_pass<64, 1>(r, sl, -m_l2, valid) : exp_pass<32, 1>(r, sl, -m_l2, valid);
                if (cnt > 0) {
                    // P V of the previous key tile reads the P columns: it must have retired
                    if (!__all_sync(0xffffffffu, mbar_wait(&o_done[g], (cnt - 1) & 1u, abort_flag))) { ok = false; break; }
                    tc_fence_after();
                }
                tmem_st_32x16(p_addr, r);
                if (ncol > 32) tmem_st_32x16(p_addr + 16, r + 16);
                if (ncol > 64) tmem_st_32x16(p_addr + 32, r + 32);
                if (ncol > 96) tmem_st_32x16(p_addr + 48, r + 48);
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
            // which drops the rows past N.  Storing a row per lane straight to global memory cost
            // about 200 cycles per 16-byte store instruction (32 lines touched by each).
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
            const int row0 = (g ? it.q0[1] : it.q0[0]) + q * 32;
            if (lane == 0 && row0 < it.n) {
                tma_store_4d(&tmO, smem + OFF_OST + (g * 4 + q) * 4096, 0, g ? it.h[1] : it.h[0], row0, it.b);
                tma_store_commit();
            }
        }
        if (lane == 0) tma_store_wait<0>();              // every output row written before the CTA exits
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

// [B, N, H, 64] view with element strides; box = box_rows rows of one head of one sample.
bool make_tmap_qkv(rs_ctx* ctx, CUtensorMap* out, const void* base, int B, int N, int H, long long bs,
                   long long rs_, long long hs, int box_rows = 128) {
    const unsigned long long dims[4] = {64, (unsigned long long)H, (unsigned long long)N, (unsigned long long)B};
    // a dimension of extent 1 never uses its stride; give it a harmless valid one
    const unsigned long long strides[3] = {(H > 1 ? (unsigned long long)hs : 64) * 2, (N > 1 ? (unsigned long long)rs_ : 64) * 2,
                                           (B > 1 ? (unsigned long long)bs : 64) * 2};
    const unsigned int box[4] = {64, 1, (unsigned int)box_rows, 1};
    return tc_encode_cached(ctx, out, base, 4, 0, dims, strides, box, 128);
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

// How a shape with more than one query tile per head is run (host side, remembered per shape).
// Two query tiles per CTA (this file): items go to the CTAs round robin, and a pair of query tiles costs
// twice a single one, so a last round with few pairs left keeps most SMs idle for a whole pair's time.
// The tiles of the last few (sample, head)s are therefore handed out one by one where that shortens the
// longest CTA: best_hs is the count with the smallest makespan under the cost model pair = 10, single = 7
// (a query tile alone runs faster than next to another, but not twice as fast: measured).
// This kernel or the one with three query tiles per CTA (rs_attn_tc3.cu)?  Both are paced by the longest
// CTA: its items (in tenths) times the key tiles of an item, plus a cost per item; microseconds fitted to
// CUDA-event times of thirteen shapes from N = 197 to 4097 (worst error 6 % and 9 %).
AttnPlan attn_plan(long long BH, int N, int G) {
    const int nt = (N + BQ - 1) / BQ, per = (N + 2 * BQ - 1) / (2 * BQ);
    auto makespan = [&](long long hs) {
        const long long pair_items = (BH - hs) * per, singles = hs * nt, all = pair_items + singles;
        long long worst = 0;
        for (int c = 0; c < G && c < all; ++c) {          // CTA c takes items c, c + G, ...
            long long load = 0;
            for (long long w = c; w < all; w += G)
                load += w < pair_items ? (((w % per) == per - 1 && (nt & 1)) ? 7 : 10) : 7;
            if (load > worst) worst = load;
        }
        return worst;
    };
    static std::mutex memo_mu;
    static std::map<std::tuple<long long, int, int>, AttnPlan> memo;
    AttnPlan plan = {0, 0, 0};
    const auto key = std::make_tuple(BH, N, G);
    std::lock_guard<std::mutex> lock(memo_mu);
    const auto hit = memo.find(key);
    if (hit != memo.end()) return hit->second;
    long long hs_max = (2ll * G + nt - 1) / nt + 1;        // enough single tiles for two rounds
    if (hs_max > BH) hs_max = BH;
    long long best = -1;
    if (N > BQ && BH * per <= 200000) {                   // (a host loop over the items for every candidate)
        for (long long hs = 0; hs <= hs_max; ++hs) {
            const long long m = makespan(hs);
            if (best < 0 || m < best) { best = m; plan.best_hs = hs; }
        }
        int wrap3 = 0;
        const long long u3 = attn_tc3_plan(BH, N, G, &wrap3);
        const double t2 = best / 10.0 * (((N + BKV - 1) / BKV) * 1.505 + 2.51) + 2.32;
        const double t3 = u3 / 10.0 * (((N + 63) / 64) * 1.136 + 1.00) + 6.71;
        plan.three = t3 < t2;
        plan.wrap3 = wrap3;
    }
    memo[key] = plan;
    return plan;
}

cudaError_t launch_attn_tc(rs_ctx* ctx, const rs_attn_desc& d, const void* q, const void* k, const void* v,
                           void* out, const int32_t* seq_lens, cudaStream_t st) {
    if (!ctx->encode_tiled) return cudaErrorNotSupported;
    static PerDeviceOnce attr_once;   // the attribute belongs to the device current at the call
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = (cudaError_t)attr_once.run(dev, [] {
        cudaError_t a = cudaFuncSetAttribute(attn_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        if (a == cudaSuccess) a = cudaFuncSetAttribute(attn_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmem);
        return (int)a;
    });
    if (e != cudaSuccess) return e;
    CUtensorMap tmQ, tmK, tmV, tmO;
    // out is [B, N, H, 64] contiguous; a softmax warp stores its 32 rows of one head at a time
    if (!make_tmap_qkv(ctx, &tmO, out, d.B, d.N, d.H, (long long)d.N * d.H * 64, (long long)d.H * 64, 64, 32) ||
        !make_tmap_qkv(ctx, &tmQ, q, d.B, d.N, d.H, d.q_batch_stride, d.q_row_stride, d.q_head_stride) ||
        !make_tmap_qkv(ctx, &tmK, k, d.B, d.N, d.H, d.k_batch_stride, d.k_row_stride, d.k_head_stride) ||
        !make_tmap_qkv(ctx, &tmV, v, d.B, d.N, d.H, d.v_batch_stride, d.v_row_stride, d.v_head_stride))
        return cudaErrorInvalidValue;
    AttnArgs args;
    args.out = (__nv_bfloat16*)out;
    args.N = d.N; args.H = d.H;
    args.dual = d.N <= BQ ? 1 : 0;
    args.per = args.dual ? (d.H + 1) / 2 : (d.N + 2 * BQ - 1) / (2 * BQ);
    long long items = (long long)args.per * (args.dual ? d.B : (long long)d.B * d.H);
    if (items >= (1ll << 30)) return cudaErrorInvalidValue;
    args.n_pair_items = (int)items; args.first_single_bh = d.B * d.H; args.tile_count = (d.N + BQ - 1) / BQ;
    if (!args.dual) {
        const long long BH = (long long)d.B * d.H;
        const int nt = args.tile_count, per = args.per;
        const AttnPlan plan = attn_plan(BH, d.N, ctx->sm_count);
        const int force = ctx->attn_kernel;                    // RS_ATTN_KERNEL=2 / 3: one kernel for every shape it takes
        if (!seq_lens && (force == 3 || (force != 2 && plan.three))) {
            CUtensorMap tmK3, tmV3;
            if (!make_tmap_qkv(ctx, &tmK3, k, d.B, d.N, d.H, d.k_batch_stride, d.k_row_stride, d.k_head_stride, 64) ||
                !make_tmap_qkv(ctx, &tmV3, v, d.B, d.N, d.H, d.v_batch_stride, d.v_row_stride, d.v_head_stride, 64))
                return cudaErrorInvalidValue;
            return launch_attn_tc3(ctx, d, tmQ, tmK3, tmV3, tmO, plan.wrap3, st);
        }
        const long long best_hs = plan.best_hs;
        args.n_pair_items = (int)((BH - best_hs) * per);
        args.first_single_bh = (int)(BH - best_hs);
        items = (BH - best_hs) * per + best_hs * nt;
    }
    args.n_items = (int)items;
    const float scale = d.scale != 0.f ? d.scale : 0.125f;
    args.scale_log2 = scale * 1.4426950408889634f;
    args.lens = seq_lens;
    args.status = ctx->d_status;
    // One resident CTA per SM walks the item list, so set-up, loads and epilogues overlap across
    // items (also for long items: measured 2-5 % over one CTA per item at N = 2305 ... 4097).
    const int nkv = (d.N + BKV - 1) / BKV;
    const int grid = args.n_items < ctx->sm_count ? args.n_items : ctx->sm_count;
    // a partial key tile is worth its own code when it is a good part of the sequence
    if (nkv <= 12) return launch_pdl(attn_tc_kernel<true>, dim3(grid), dim3(kThreads), kSmem, st, tmQ, tmK, tmV, tmO, args);
    return launch_pdl(attn_tc_kernel<false>, dim3(grid), dim3(kThreads), kSmem, st, tmQ, tmK, tmV, tmO, args);
}

}  // namespace rs
