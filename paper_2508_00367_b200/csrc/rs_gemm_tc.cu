// bf16 GEMM on the 5th-generation tensor cores with the block's epilogues fused in:
//     out[M, N] = epilogue(A[M, K] . W[N, K]^T)
// A and W are K-major; TMA (128-byte swizzle) feeds a shared-memory ring, one thread
// issues tcgen05.mma into a double-buffered fp32 accumulator in tensor memory, and eight
// epilogue warps drain it with tcgen05.ld while the next tile's main loop runs.
//
// Epilogues (Eq. att, Eq. MLP, Sec. 3.2):
//   EPI_BIAS       out = acc + b                          -> bf16      (QKV projection)
//   EPI_BIAS_GELU  out = GELU(acc + b)                    -> bf16      (FC1)
//   EPI_RESID      out = acc + b + x                      -> fp32      (projection + residual = x')
//   EPI_SCORE      m = acc + b;  out = m + x';  partial sums of (m - x')^2 (or m^2) per row
//                                                          -> bf16/fp32 (FC2 + residual + shift score)
#include "rs_internal.h"
#include "rs_tc.cuh"

namespace rs {

namespace {

using namespace tc;

enum { EPI_BIAS = 0, EPI_BIAS_GELU = 1, EPI_RESID = 2, EPI_SCORE = 3 };

constexpr int BM = 128, BK = 64;
constexpr int kThreads = 320;                 // warp 0: TMA, warp 1: MMA, warps 2-9: epilogue
constexpr int kEpiWarps = 8;
constexpr int A_BYTES = BM * BK * 2;          // 16 KB

template <int BN> struct Cfg {
    static constexpr int B_BYTES = BN * BK * 2;
    static constexpr int STAGES = (BN == 128) ? 6 : 4;
    static constexpr int STAGE_BYTES = A_BYTES + B_BYTES;
    static constexpr int TMEM_COLS = 2 * BN;
    static constexpr size_t SMEM = (size_t)STAGES * STAGE_BYTES + 1024 /*align slack*/ + 256 /*barriers*/;
};

struct GemmArgs {
    int M, N, K;
    const float* bias;        // [N] or null
    const void* residual;     // EPI_RESID: bf16 [M, N];  EPI_SCORE: fp32 [M, N]
    void* out;                // [M, N]
    float* partials;          // EPI_SCORE: [M, 2 * N / BN] sums of squares
    int score_delta;          // EPI_SCORE: 1 => sum m^2 instead of (m - x')^2
    int* status;
};

__device__ __forceinline__ float gelu_erf(float v) {
    return 0.5f * v * (1.f + erff(v * 0.70710678118654752f));
}

__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}

template <int BN, int EPI, typename OutT>
__global__ void __launch_bounds__(kThreads, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const GemmArgs args) {
    using C = Cfg<BN>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint64_t* bars = reinterpret_cast<uint64_t*>(smem + (size_t)C::STAGES * C::STAGE_BYTES);
    uint64_t* full = bars;                       // [STAGES]
    uint64_t* empty = bars + C::STAGES;          // [STAGES]
    uint64_t* tfull = bars + 2 * C::STAGES;      // [2]
    uint64_t* tempty = bars + 2 * C::STAGES + 2; // [2]
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * C::STAGES + 4);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int num_m = (args.M + BM - 1) / BM, num_n = args.N / BN;
    const int tiles = num_m * num_n, kblocks = args.K / BK;

    if (threadIdx.x == 0) {
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
        for (int s = 0; s < C::STAGES; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
        for (int a = 0; a < 2; ++a) { mbar_init(&tfull[a], 1); mbar_init(&tempty[a], kEpiWarps); }
        *abort_flag = 0;
        mbar_fence_init();
    }
    if (warp == 1) {
        tmem_alloc(tmem_slot, C::TMEM_COLS);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        // ---------------- TMA producer ----------------
        if (elect_one()) {
            uint32_t it = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
                const int m0 = (tile / num_n) * BM, n0 = (tile % num_n) * BN;
                for (int kb = 0; kb < kblocks; ++kb, ++it) {
                    const int s = it % C::STAGES;
                    const uint32_t ph = (it / C::STAGES) & 1u;
                    if (!mbar_wait(&empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                    uint8_t* sa = smem + (size_t)s * C::STAGE_BYTES;
                    mbar_expect_tx(&full[s], C::STAGE_BYTES);
                    tma_load_2d(sa, &tmA, &full[s], kb * BK, m0);
                    tma_load_2d(sa + A_BYTES, &tmB, &full[s], kb * BK, n0);
                }
            }
            // Copies this thread started must have landed before the CTA may exit.
            const uint32_t issued = it;
            for (int s = 0; s < C::STAGES; ++s) {
                if ((uint32_t)s >= issued) break;
                const uint32_t last = ((issued - 1 - s) / C::STAGES) * C::STAGES + s;   // last use of stage s
                mbar_wait(&full[s], (last / C::STAGES) & 1u, abort_flag);
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------
        if (elect_one()) {
            constexpr uint32_t idesc = idesc_bf16(BM, BN, 0, 0);
            uint32_t it = 0, tl = 0;
            bool ok = true;
            for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
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
                        mma_ss(d_tmem, da + 2u * k, db + 2u * k, idesc, (kb | k) != 0);
                    mma_commit(&empty[s]);              // frees the stage when these MMAs retire
                }
                if (ok) mma_commit(&tfull[a]);          // accumulator complete
            }
        }
    } else {
        // ---------------- epilogue ----------------
        const int q = warp & 3;                          // TMEM lane quadrant this warp may read
        const int half = (warp - 2) >> 2;                // which half of the tile's columns
        constexpr int HALF_N = BN / 2;
        uint32_t tl = 0;
        bool ok = true;
        for (int tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tl) {
            const int m0 = (tile / num_n) * BM, nt = tile % num_n, n0 = nt * BN;
            const uint32_t a = tl & 1u, aph = (tl >> 1) & 1u;
            if (!__all_sync(0xffffffffu, mbar_wait(&tfull[a], aph, abort_flag))) { ok = false; break; }
            tc_fence_after();
            const int row = m0 + q * 32 + lane;
            const bool valid = row < args.M;
            const uint32_t taddr = tmem_base + ((uint32_t)(q * 32) << 16) + a * BN + half * HALF_N;
            float sq = 0.f;
#pragma unroll 1
            for (int c = 0; c < HALF_N; c += 32) {
                uint32_t r[32];
                __syncwarp();                            // tcgen05.ld is warp-collective
                tmem_ld_32x32(taddr + c, r);
                tmem_wait_ld();
                const int col = n0 + half * HALF_N + c;
                float v[32];
#pragma unroll
                for (int j = 0; j < 32; j += 4) {
                    float4 b = args.bias ? __ldg(reinterpret_cast<const float4*>(args.bias + col + j))
                                         : make_float4(0.f, 0.f, 0.f, 0.f);
                    v[j] = __uint_as_float(r[j]) + b.x;
                    v[j + 1] = __uint_as_float(r[j + 1]) + b.y;
                    v[j + 2] = __uint_as_float(r[j + 2]) + b.z;
                    v[j + 3] = __uint_as_float(r[j + 3]) + b.w;
                }
                if (!valid) continue;
                const size_t off = (size_t)row * args.N + col;
                if (EPI == EPI_BIAS || EPI == EPI_BIAS_GELU) {
                    if (EPI == EPI_BIAS_GELU) {
#pragma unroll
                        for (int j = 0; j < 32; ++j) v[j] = gelu_erf(v[j]);
                    }
                    uint4* o = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(args.out) + off);
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        o[j] = make_uint4(pack_bf16(v[8 * j], v[8 * j + 1]), pack_bf16(v[8 * j + 2], v[8 * j + 3]),
                                          pack_bf16(v[8 * j + 4], v[8 * j + 5]), pack_bf16(v[8 * j + 6], v[8 * j + 7]));
                } else if (EPI == EPI_RESID) {
                    const uint4* rp = reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(args.residual) + off);
                    float4* o = reinterpret_cast<float4*>(reinterpret_cast<float*>(args.out) + off);
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        const uint4 x = __ldg(rp + j);
                        const uint32_t w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            v[8 * j + 2 * e] += __uint_as_float(w[e] << 16);
                            v[8 * j + 2 * e + 1] += __uint_as_float(w[e] & 0xffff0000u);
                        }
                        o[2 * j] = make_float4(v[8 * j], v[8 * j + 1], v[8 * j + 2], v[8 * j + 3]);
                        o[2 * j + 1] = make_float4(v[8 * j + 4], v[8 * j + 5], v[8 * j + 6], v[8 * j + 7]);
                    }
                } else {   // EPI_SCORE
                    const float4* rp = reinterpret_cast<const float4*>(reinterpret_cast<const float*>(args.residual) + off);
#pragma unroll
                    for (int j = 0; j < 8; ++j) {
                        const float4 x = __ldg(rp + j);
                        const float xs[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
                        for (int e = 0; e < 4; ++e) {
                            const float m = v[4 * j + e];
                            const float d = args.score_delta ? m : m - xs[e];
                            sq = fmaf(d, d, sq);
                            v[4 * j + e] = m + xs[e];
                        }
                    }
                    if (sizeof(OutT) == 4) {
                        float4* o = reinterpret_cast<float4*>(reinterpret_cast<float*>(args.out) + off);
#pragma unroll
                        for (int j = 0; j < 8; ++j) o[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
                    } else {
                        uint4* o = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(args.out) + off);
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            o[j] = make_uint4(pack_bf16(v[8 * j], v[8 * j + 1]), pack_bf16(v[8 * j + 2], v[8 * j + 3]),
                                              pack_bf16(v[8 * j + 4], v[8 * j + 5]), pack_bf16(v[8 * j + 6], v[8 * j + 7]));
                    }
                }
            }
            if (EPI == EPI_SCORE && valid)
                args.partials[(size_t)row * (2 * num_n) + 2 * nt + half] = sq;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&tempty[a]);
        }
    }

    __syncthreads();
    if (*abort_flag && threadIdx.x == 0) atomicExch(args.status, RS_DEV_TIMEOUT);
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, C::TMEM_COLS);
    }
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

template <int BN, int EPI, typename OutT>
cudaError_t launch_one(const CUtensorMap& tmA, const CUtensorMap& tmB, const GemmArgs& args, int sm_count,
                       cudaStream_t st) {
    using C = Cfg<BN>;
    static bool attr_done = false;   // per instantiation; the attribute is per function, set once
    if (!attr_done) {
        cudaError_t e = cudaFuncSetAttribute(gemm_tc_kernel<BN, EPI, OutT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             (int)C::SMEM);
        if (e != cudaSuccess) return e;
        attr_done = true;
    }
    const int tiles = ((args.M + BM - 1) / BM) * (args.N / BN);
    const int grid = tiles < sm_count ? tiles : sm_count;
    gemm_tc_kernel<BN, EPI, OutT><<<grid, kThreads, C::SMEM, st>>>(tmA, tmB, args);
    return cudaGetLastError();
}

}  // namespace

void* tc_get_encode_fn() {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPointByVersion("cuTensorMapEncodeTiled", &fn, 12000, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess)
        return nullptr;
    return fn;
}

// Tensor map over a row-major bf16 matrix [rows, cols] (cols contiguous), box [box_rows, 64], 128-byte swizzle.
bool tc_make_tmap_2d(void* encode_fn, CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols,
                     uint64_t row_stride_elems, uint32_t box_rows) {
    EncodeTiledFn fn = reinterpret_cast<EncodeTiledFn>(encode_fn);
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {row_stride_elems * 2};
    const cuuint32_t box[2] = {64, box_rows};
    const cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
              CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

bool gemm_tc_supported(long long M, int N, int K) {
    return M >= 1 && M < (1ll << 31) && N >= 128 && (N % 128) == 0 && K >= 64 && (K % 64) == 0;
}

int gemm_tc_score_parts(int N) {   // partial sums per row written by the EPI_SCORE epilogue
    const int bn = 128;
    return 2 * (N / bn);
}

cudaError_t launch_gemm_tc(rs_ctx* ctx, int epi, const void* A, const void* W, const float* bias,
                           const void* residual, void* out, rs_dtype out_dtype, float* partials, int score_delta,
                           long long M, int N, int K, cudaStream_t st) {
    if (!ctx->encode_tiled) return cudaErrorNotSupported;
    // Tile width: the score epilogue indexes its partial sums by 128-column tiles; elsewhere pick the
    // width with fewer, fuller waves over the SMs.
    int bn = 128;
    if (epi != EPI_SCORE && (N % 256) == 0) {
        const long long mt = (M + BM - 1) / BM;
        const long long w128 = (mt * (N / 128) + ctx->sm_count - 1) / ctx->sm_count * 128;
        const long long w256 = (mt * (N / 256) + ctx->sm_count - 1) / ctx->sm_count * 256;
        if (w256 <= w128) bn = 256;
    }
    CUtensorMap tmA, tmB;
    if (!tc_make_tmap_2d(ctx->encode_tiled, &tmA, A, (uint64_t)M, (uint64_t)K, (uint64_t)K, BM) ||
        !tc_make_tmap_2d(ctx->encode_tiled, &tmB, W, (uint64_t)N, (uint64_t)K, (uint64_t)K, (uint32_t)bn))
        return cudaErrorInvalidValue;
    GemmArgs args;
    args.M = (int)M; args.N = N; args.K = K; args.bias = bias; args.residual = residual; args.out = out;
    args.partials = partials; args.score_delta = score_delta; args.status = ctx->d_status;
    const int sms = ctx->sm_count;
    switch (epi) {
        case EPI_BIAS:
            return bn == 256 ? launch_one<256, EPI_BIAS, __nv_bfloat16>(tmA, tmB, args, sms, st)
                             : launch_one<128, EPI_BIAS, __nv_bfloat16>(tmA, tmB, args, sms, st);
        case EPI_BIAS_GELU:
            return bn == 256 ? launch_one<256, EPI_BIAS_GELU, __nv_bfloat16>(tmA, tmB, args, sms, st)
                             : launch_one<128, EPI_BIAS_GELU, __nv_bfloat16>(tmA, tmB, args, sms, st);
        case EPI_RESID:
            return bn == 256 ? launch_one<256, EPI_RESID, float>(tmA, tmB, args, sms, st)
                             : launch_one<128, EPI_RESID, float>(tmA, tmB, args, sms, st);
        case EPI_SCORE:
            return out_dtype == RS_F32 ? launch_one<128, EPI_SCORE, float>(tmA, tmB, args, sms, st)
                                       : launch_one<128, EPI_SCORE, __nv_bfloat16>(tmA, tmB, args, sms, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace rs
