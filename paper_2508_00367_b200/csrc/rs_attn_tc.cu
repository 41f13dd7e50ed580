// Fused attention on the tensor cores (Eq. sa): out = Softmax(Q K^T * scale) V per
// (sample, head), head dimension 64, without ever writing the N x N matrix.
//
// One CTA owns 128 query rows of one (sample, head) and streams the keys/values in tiles
// of 128 through a two-stage TMA ring.  Per tile:  S = Q K^T  (tcgen05.mma, fp32 in tensor
// memory)  ->  four softmax warps (one row per thread) keep the running max / sum, rescale
// the O accumulator when the max moves, and write P = exp2(S*c - m*c) as bf16 into shared
// memory in the K-major 128-byte-swizzled operand layout  ->  O += P V  (tcgen05.mma, V
// used as an MN-major operand straight from its TMA tile).  Two CTAs share an SM so one
// CTA's softmax overlaps the other's MMAs.  The first 64 columns of P reuse the K tile's
// buffer, which is dead once S has been computed.
#include <math.h>

#include "rs_internal.h"
#include "rs_tc.cuh"

namespace rs {

namespace {

using namespace tc;

constexpr int BQ = 128, BKV = 128, DH = 64;
constexpr int TILE_BYTES = 128 * DH * 2;        // 16 KB: a [128, 64] bf16 tile
constexpr int kThreads = 192;                   // warp 0: TMA, warp 1: MMA, warps 2-5: softmax
constexpr int kTmemCols = 256;                  // S: columns 0..127, O: columns 128..191
constexpr int kOCol = 128;
// shared memory: Q | K0 | K1 | V0 | V1 | P-high | barriers
constexpr int OFF_Q = 0, OFF_K = TILE_BYTES, OFF_V = 3 * TILE_BYTES, OFF_P1 = 5 * TILE_BYTES;
constexpr int OFF_BAR = 6 * TILE_BYTES;
constexpr size_t kSmem = (size_t)OFF_BAR + 128 + 1024 /*alignment slack*/;

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

__global__ void __launch_bounds__(kThreads, 2)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK,
               const __grid_constant__ CUtensorMap tmV, const AttnArgs args) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
    uint64_t* bar_q = bars;            // Q tile landed
    uint64_t* kv_full = bars + 1;      // [2] K and V tile landed
    uint64_t* kv_empty = bars + 3;     // [2] stage free again (O += P V retired)
    uint64_t* s_full = bars + 5;       // S tile complete in tensor memory
    uint64_t* p_ready = bars + 6;      // P written, O rescaled, S consumed (128 arrivals)
    uint64_t* o_done = bars + 7;       // O += P V retired
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int N = args.N;
    const int q0 = blockIdx.x * BQ, h = blockIdx.y, b = blockIdx.z;
    const int nkv = (N + BKV - 1) / BKV;

    if (threadIdx.x == 0) {
        prefetch_tmap(&tmQ); prefetch_tmap(&tmK); prefetch_tmap(&tmV);
        mbar_init(bar_q, 1);
        for (int s = 0; s < 2; ++s) { mbar_init(&kv_full[s], 1); mbar_init(&kv_empty[s], 1); }
        mbar_init(s_full, 1);
        mbar_init(p_ready, 128);
        mbar_init(o_done, 1);
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            mbar_expect_tx(bar_q, TILE_BYTES);
            tma_load_4d(smem + OFF_Q, &tmQ, bar_q, 0, h, q0, b);
            int issued = 0;
            for (int j = 0; j < nkv; ++j, ++issued) {
                const int s = j & 1;
                if (!mbar_wait(&kv_empty[s], ((j >> 1) & 1) ^ 1, abort_flag)) break;
                mbar_expect_tx(&kv_full[s], 2 * TILE_BYTES);
                tma_load_4d(smem + OFF_K + s * TILE_BYTES, &tmK, &kv_full[s], 0, h, j * BKV, b);
                tma_load_4d(smem + OFF_V + s * TILE_BYTES, &tmV, &kv_full[s], 0, h, j * BKV, b);
            }
            // every copy started here must have landed before the CTA exits
            mbar_wait(bar_q, 0, abort_flag);
            for (int s = 0; s < 2 && s < issued; ++s) {
                const int last = ((issued - 1 - s) / 2) * 2 + s;
                mbar_wait(&kv_full[s], (last >> 1) & 1, abort_flag);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            bool ok = mbar_wait(bar_q, 0, abort_flag);
            tc_fence_after();
            const uint32_t sq = smem_u32(smem + OFF_Q);
            for (int j = 0; j < nkv && ok; ++j) {
                const int s = j & 1;
                const int valid = min(BKV, N - j * BKV);
                const int n_s = (valid + 15) & ~15;           // S columns actually needed
                const int ksteps = (valid + 15) >> 4;         // 16-key slabs of P V actually needed
                if (!mbar_wait(&kv_full[s], (j >> 1) & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t sk = smem_u32(smem + OFF_K + s * TILE_BYTES);
                const uint32_t sv = smem_u32(smem + OFF_V + s * TILE_BYTES);
                // S = Q K^T : both operands K-major (head dimension contiguous)
                const uint32_t idesc_s = idesc_bf16(BQ, n_s, 0, 0);
                const uint64_t dq = smem_desc_sw128(sq, 16, 1024);
                const uint64_t dk = smem_desc_sw128(sk, 16, 1024);
#pragma unroll
                for (int k = 0; k < DH / 16; ++k) mma_ss(tmem_base, dq + 2u * k, dk + 2u * k, idesc_s, k != 0);
                mma_commit(s_full);
                // O += P V : P K-major from shared memory (first 64 keys in the K buffer, rest in P-high),
                // V MN-major (head dimension contiguous), 16 keys = 2048 bytes per slab.
                if (!mbar_wait(p_ready, j & 1, abort_flag)) { ok = false; break; }
                tc_fence_after();
                const uint32_t idesc_o = idesc_bf16(BQ, DH, 0, 1);
                const uint32_t sp1 = smem_u32(smem + OFF_P1);
                for (int k = 0; k < ksteps; ++k) {
                    const uint32_t pa = (k < 4 ? sk : sp1) + (uint32_t)(k & 3) * 32u;
                    const uint64_t dp = smem_desc_sw128(pa, 16, 1024);
                    const uint64_t dv = smem_desc_sw128(sv + (uint32_t)k * 2048u, 16, 1024);
                    mma_ss(tmem_base + kOCol, dp, dv, idesc_o, (j | k) != 0);
                }
                mma_commit(&kv_empty[s]);
                mma_commit(o_done);
            }
        }
    } else {
        // ---------------- softmax / correction / epilogue: one query row per thread ----------------
        const int q = warp & 3;
        const int row = q0 + q * 32 + lane;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(q * 32) << 16);
        const float sl = args.scale_log2;
        const int r8 = (q * 32 + lane) & 7;
        const uint32_t row_off = (uint32_t)((q * 32 + lane) >> 3) * 1024u + (uint32_t)r8 * 128u;
        float m_run = -INFINITY, l_run = 0.f;
        bool ok = true;
        for (int j = 0; j < nkv && ok; ++j) {
            const int s = j & 1;
            const int valid = min(BKV, N - j * BKV);
            const int nchunks = (valid + 31) >> 5;
            // the warp moves as one through the collective tensor-memory loads below
            if (!__all_sync(0xffffffffu, mbar_wait(s_full, j & 1, abort_flag))) { ok = false; break; }
            tc_fence_after();
            // pass 1: row maximum over the valid keys
            float mx = m_run;
            for (int c = 0; c < nchunks; ++c) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld_32x32(lane_addr + c * 32, r);
                tmem_wait_ld();
                const int lim = valid - c * 32;
#pragma unroll
                for (int i = 0; i < 32; ++i) mx = fmaxf(mx, i < lim ? __uint_as_float(r[i]) : -INFINITY);
            }
            const float alpha = ex2((m_run - mx) * sl);   // 0 on the first tile (m_run = -inf)
            const float mneg = -mx * sl;
            l_run *= alpha;
            m_run = mx;
            if (j > 0) {
                // the previous O += P V must have retired before O is rescaled and P-high is overwritten
                if (!__all_sync(0xffffffffu, mbar_wait(o_done, (j - 1) & 1, abort_flag))) { ok = false; break; }
                tc_fence_after();
                if (__any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll
                    for (int c = 0; c < 2; ++c) {
                        uint32_t r[32];
                        tmem_ld_32x32(lane_addr + kOCol + c * 32, r);
                        tmem_wait_ld();
#pragma unroll
                        for (int i = 0; i < 32; ++i) r[i] = __float_as_uint(__uint_as_float(r[i]) * alpha);
                        tmem_st_32x32(lane_addr + kOCol + c * 32, r);
                    }
                    tmem_wait_st();
                }
            }
            // pass 2: P = exp2(S*c - m*c) -> bf16 -> shared memory (K-major, 128-byte swizzle)
            uint8_t* p_lo = smem + OFF_K + s * TILE_BYTES;
            uint8_t* p_hi = smem + OFF_P1;
            for (int c = 0; c < nchunks; ++c) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld_32x32(lane_addr + c * 32, r);
                tmem_wait_ld();
                const int lim = valid - c * 32;
                uint32_t pk[16];
#pragma unroll
                for (int i = 0; i < 32; i += 2) {
                    const float p0 = i < lim ? ex2(fmaf(__uint_as_float(r[i]), sl, mneg)) : 0.f;
                    const float p1 = i + 1 < lim ? ex2(fmaf(__uint_as_float(r[i + 1]), sl, mneg)) : 0.f;
                    l_run += p0 + p1;
                    pk[i >> 1] = pack_bf16(p0, p1);
                }
                uint8_t* base = (c < 2 ? p_lo : p_hi) + row_off;
#pragma unroll
                for (int g = 0; g < 4; ++g) {                 // four 16-byte groups of 8 keys
                    const int chunk16 = (c & 1) * 4 + g;      // position inside the 128-byte row
                    *reinterpret_cast<uint4*>(base + ((chunk16 ^ r8) << 4)) =
                        make_uint4(pk[4 * g], pk[4 * g + 1], pk[4 * g + 2], pk[4 * g + 3]);
                }
            }
            fence_async_smem();
            tc_fence_before();
            mbar_arrive(p_ready);
        }
        // epilogue: O / l -> bf16 -> global
        if (ok && __all_sync(0xffffffffu, mbar_wait(o_done, (nkv - 1) & 1, abort_flag))) {
            tc_fence_after();
            const float inv = 1.f / l_run;
            __nv_bfloat16* op = args.out + ((size_t)((size_t)b * N + row) * args.H + h) * DH;
#pragma unroll
            for (int c = 0; c < 2; ++c) {
                uint32_t r[32];
                __syncwarp();
                tmem_ld_32x32(lane_addr + kOCol + c * 32, r);
                tmem_wait_ld();
                if (row < N) {
#pragma unroll
                    for (int g = 0; g < 4; ++g) {
                        uint32_t w[4];
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            w[e] = pack_bf16(__uint_as_float(r[8 * g + 2 * e]) * inv, __uint_as_float(r[8 * g + 2 * e + 1]) * inv);
                        *reinterpret_cast<uint4*>(op + c * 32 + g * 8) = make_uint4(w[0], w[1], w[2], w[3]);
                    }
                }
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicExch(args.status, RS_DEV_TIMEOUT);
    if (warp == 1) {
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
    const dim3 grid((d.N + BQ - 1) / BQ, d.H, d.B);
    attn_tc_kernel<<<grid, kThreads, kSmem, st>>>(tmQ, tmK, tmV, args);
    return cudaGetLastError();
}

}  // namespace rs
