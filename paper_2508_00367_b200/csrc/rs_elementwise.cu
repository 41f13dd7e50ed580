// HBM-bound row kernels: LayerNorm, the representation-shift score (Sec. 3.2)
// and the residual-add epilogue with the score fused in.  One warp owns one
// token row; rows move as 16-byte vectors, several in flight per lane.
#include "rs_internal.h"
#include "rs_device.cuh"

namespace rs {

namespace {

constexpr int kWarpsPerCta = 8;

// ---------------------------------------------------------------- LayerNorm
// LN of Eq. att / Eq. MLP: mean and biased variance over D, then affine.  One warp per row; the
// row stays in registers as packed 16-byte pieces (unpacked once per pass over it), which keeps
// the kernel at 48 to 64 registers so that four or five CTAs per SM cover the memory latency.
template <typename TI, typename TO, int MAXV>
__global__ void __launch_bounds__(kWarpsPerCta * 32, MAXV <= 4 ? 5 : 4)
layernorm_kernel(const TI* __restrict__ x, const float* __restrict__ gamma,
                 const float* __restrict__ beta, float eps, long long T, int D, TO* __restrict__ out,
                 const int32_t* __restrict__ row_map) {
    constexpr int VN = Vec16<TI>::N;
    grid_dep_launch();
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    if (row >= T) return;
    const int nvec = D / VN;
    const long long src = row_map ? (long long)row_map[row] : row;
    const uint4* xr = reinterpret_cast<const uint4*>(x + src * D);
    uint4 raw[MAXV];
#pragma unroll
    for (int j = 0; j < MAXV; ++j) {
        const int iv = j * 32 + lane;
        if (iv < nvec) raw[j] = ld_stream(xr + iv);
    }
    layernorm_row<TI, TO, MAXV>(raw, nvec, lane, gamma, beta, eps, D, out + row * D);
}

// ---------------------------------------------------------------- shift score
// s = D(F(x), x) per token (Sec. 3.2); DIST 0: L2, 1: L1, 2: cosine distance.
// One warp per token.  The 16-byte pieces stay packed in registers until they are reduced, so
// that eight loads per lane are in flight at about 48 registers per thread and enough warps
// fit an SM to cover the HBM latency.
template <typename T, int DIST>
__global__ void __launch_bounds__(kWarpsPerCta * 32, 5)
shift_score_kernel(const T* __restrict__ after, const T* __restrict__ before, long long rows, int D,
                   float* __restrict__ scores) {
    constexpr int VN = Vec16<T>::N;
    constexpr int UNROLL = 4;
    grid_dep_launch();
    grid_dep_wait();
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int nvec = D / VN;
    const uint4* a = reinterpret_cast<const uint4*>(after + row * D);
    const uint4* b = reinterpret_cast<const uint4*>(before + row * D);
    float acc = 0.f, aa = 0.f, bb = 0.f;
    for (int base = 0; base < nvec; base += 32 * UNROLL) {
        uint4 ra[UNROLL], rb[UNROLL];
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int iv = base + u * 32 + lane;
            if (iv < nvec) { ra[u] = ld_stream(a + iv); rb[u] = ld_stream(b + iv); }
        }
#pragma unroll
        for (int u = 0; u < UNROLL; ++u) {
            const int iv = base + u * 32 + lane;
            if (iv < nvec) {
                float va[VN], vb[VN];
                unpack16<T>(ra[u], va);
                unpack16<T>(rb[u], vb);
#pragma unroll
                for (int e = 0; e < VN; ++e) {
                    if (DIST == 0) { const float d = va[e] - vb[e]; acc = fmaf(d, d, acc); }
                    else if (DIST == 1) { acc += fabsf(va[e] - vb[e]); }
                    else {
                        acc = fmaf(va[e], vb[e], acc);
                        aa = fmaf(va[e], va[e], aa);
                        bb = fmaf(vb[e], vb[e], bb);
                    }
                }
            }
        }
    }
    acc = warp_sum(acc);
    float s;
    if (DIST == 0) s = sqrtf(acc);
    else if (DIST == 1) s = acc;
    else {
        aa = warp_sum(aa); bb = warp_sum(bb);
        s = 1.f - acc / fmaxf(sqrtf(aa) * sqrtf(bb), 1e-12f);
    }
    if (lane == 0) scores[row] = s;
}

// ---------------------------------------------------------------- residual add + score
// x_hat = m + x' and the score of the chosen pair of representations (Sec. 3.3 "Operation
// choice"): MODE 0 |m - x'| (ii), 1 |m|, 2 |SA(LN(x)) - x| = |x' - 2x| (i), 3 |x_hat - x| (iii).
// The score rides on the residual-add pass, which already has the operands in registers.
template <typename TO, typename TX, int MODE>
__global__ void __launch_bounds__(kWarpsPerCta * 32)
residual_score_kernel(const float* __restrict__ m, const float* __restrict__ xp, const TX* __restrict__ x0,
                      long long rows, int D, int dist, TO* __restrict__ x_hat, float* __restrict__ scores) {
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * kWarpsPerCta + (threadIdx.x >> 5);
    if (row >= rows) return;
    const int nvec = D / 4;
    float acc = 0.f, uu = 0.f, vv = 0.f;
    for (int iv = lane; iv < nvec; iv += 32) {
        const float4 a = *reinterpret_cast<const float4*>(m + row * D + iv * 4);
        const float4 b = *reinterpret_cast<const float4*>(xp + row * D + iv * 4);
        const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
        float y[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            y[e] = av[e] + bv[e];
            float u, v;                              // the scored pair
            if (MODE == 0) { u = av[e]; v = bv[e]; }
            else if (MODE == 1) { u = y[e]; v = bv[e]; }
            else {
                const float x = to_float(x0[row * D + iv * 4 + e]);
                u = MODE == 2 ? bv[e] - x : y[e];    // SA(LN(x)) = x' - x
                v = x;
            }
            if (dist == RS_DIST_L2) { const float d = u - v; acc = fmaf(d, d, acc); }
            else if (dist == RS_DIST_L1) acc += fabsf(u - v);
            else { acc = fmaf(u, v, acc); uu = fmaf(u, u, uu); vv = fmaf(v, v, vv); }
        }
        store_n<TO, 4>(x_hat + row * D + iv * 4, y);
    }
    acc = warp_sum(acc);
    float sc = dist == RS_DIST_L2 ? sqrtf(acc) : acc;
    if (dist == RS_DIST_COS) {
        uu = warp_sum(uu); vv = warp_sum(vv);
        sc = 1.f - acc / fmaxf(sqrtf(uu) * sqrtf(vv), 1e-12f);
    }
    if (lane == 0 && scores) scores[row] = sc;
}

inline unsigned row_grid(long long rows) { return (unsigned)((rows + kWarpsPerCta - 1) / kWarpsPerCta); }

template <typename TI, typename TO>
cudaError_t ln_dispatch(const void* x, const float* g, const float* b, float eps, long long T, int D,
                        void* out, const int32_t* row_map, cudaStream_t st) {
    const int nvec = D / Vec16<TI>::N;
    const dim3 grid(row_grid(T)), block(kWarpsPerCta * 32);
    if (nvec <= 32 * 4)
        return launch_pdl(layernorm_kernel<TI, TO, 4>, grid, block, 0, st, (const TI*)x, g, b, eps, T, D, (TO*)out, row_map);
    else if (nvec <= 32 * 8)
        return launch_pdl(layernorm_kernel<TI, TO, 8>, grid, block, 0, st, (const TI*)x, g, b, eps, T, D, (TO*)out, row_map);
    return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_layernorm(rs_dtype in_dtype, rs_dtype out_dtype, const void* x, const float* gamma,
                             const float* beta, float eps, long long T, int D, void* out,
                             const int32_t* row_map, cudaStream_t st) {
    if (T == 0) return cudaSuccess;
    if (in_dtype == RS_F32 && out_dtype == RS_F32) return ln_dispatch<float, float>(x, gamma, beta, eps, T, D, out, row_map, st);
    if (in_dtype == RS_F32 && out_dtype == RS_BF16) return ln_dispatch<float, __nv_bfloat16>(x, gamma, beta, eps, T, D, out, row_map, st);
    if (in_dtype == RS_BF16 && out_dtype == RS_BF16) return ln_dispatch<__nv_bfloat16, __nv_bfloat16>(x, gamma, beta, eps, T, D, out, row_map, st);
    return ln_dispatch<__nv_bfloat16, float>(x, gamma, beta, eps, T, D, out, row_map, st);
}

cudaError_t launch_shift_score(rs_dtype dtype, rs_dist dist, long long T, int D, const void* after,
                               const void* before, float* scores, cudaStream_t st) {
    if (T == 0) return cudaSuccess;
    const dim3 grid(row_grid(T)), block(kWarpsPerCta * 32);
#define RS_SCORE_CASE(TT, DD)                                                                   \
    return launch_pdl(shift_score_kernel<TT, DD>, grid, block, 0, st, (const TT*)after, (const TT*)before, T, D, scores)
    if (dtype == RS_BF16) {
        if (dist == RS_DIST_L2) RS_SCORE_CASE(__nv_bfloat16, 0);
        else if (dist == RS_DIST_L1) RS_SCORE_CASE(__nv_bfloat16, 1);
        else RS_SCORE_CASE(__nv_bfloat16, 2);
    } else {
        if (dist == RS_DIST_L2) RS_SCORE_CASE(float, 0);
        else if (dist == RS_DIST_L1) RS_SCORE_CASE(float, 1);
        else RS_SCORE_CASE(float, 2);
    }
#undef RS_SCORE_CASE
    return cudaGetLastError();
}

cudaError_t launch_residual_score(const float* m, const float* x_prime, const void* x, rs_dtype x_dtype,
                                  long long T, int D, rs_score_mode mode, rs_dist dist, rs_dtype out_dtype,
                                  void* x_hat, float* scores, cudaStream_t st) {
    if (T == 0) return cudaSuccess;
    const dim3 grid(row_grid(T)), block(kWarpsPerCta * 32);
#define RS_RES_CASE(TO, TX, MD)                                                                                  \
    residual_score_kernel<TO, TX, MD><<<grid, block, 0, st>>>(m, x_prime, (const TX*)x, T, D, (int)dist, (TO*)x_hat, scores)
#define RS_RES_MODE(TO, TX)                                     \
    do {                                                        \
        if (mode == RS_SCORE_MLP) RS_RES_CASE(TO, TX, 0);       \
        else if (mode == RS_SCORE_MLP_DELTA) RS_RES_CASE(TO, TX, 1); \
        else if (mode == RS_SCORE_ATTN) RS_RES_CASE(TO, TX, 2); \
        else RS_RES_CASE(TO, TX, 3);                            \
    } while (0)
    if (out_dtype == RS_BF16) {
        if (x_dtype == RS_BF16) RS_RES_MODE(__nv_bfloat16, __nv_bfloat16); else RS_RES_MODE(__nv_bfloat16, float);
    } else {
        if (x_dtype == RS_BF16) RS_RES_MODE(float, __nv_bfloat16); else RS_RES_MODE(float, float);
    }
#undef RS_RES_MODE
#undef RS_RES_CASE
    return cudaGetLastError();
}

// LayerNorm folded into the projection that follows: one warp per output row n of W [n_out, K].
namespace {
__global__ void __launch_bounds__(256)
ln_fold_prep_kernel(const __nv_bfloat16* __restrict__ W, const float* __restrict__ bias, const float* __restrict__ g,
                    const float* __restrict__ beta, int n_out, int K, __nv_bfloat16* __restrict__ w_out,
                    float* __restrict__ c_out, float* __restrict__ b_out) {
    const int n = blockIdx.x * 8 + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (n >= n_out) return;
    float c = 0.f, bb = 0.f;
    for (int k = lane; k < K; k += 32) {
        const float w = __bfloat162float(W[(size_t)n * K + k]);
        const __nv_bfloat16 ws = __float2bfloat16_rn(w * g[k]);
        w_out[(size_t)n * K + k] = ws;
        c += __bfloat162float(ws);
        bb = fmaf(w, beta[k], bb);
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        c += __shfl_xor_sync(0xffffffffu, c, o);
        bb += __shfl_xor_sync(0xffffffffu, bb, o);
    }
    if (lane == 0) {
        c_out[n] = c;
        b_out[n] = bb + (bias ? bias[n] : 0.f);
    }
}
}  // namespace

cudaError_t launch_ln_fold_prep(const void* W, const float* bias, const float* g, const float* beta, int n_out, int K,
                                void* w_out, float* c_out, float* b_out, cudaStream_t st) {
    ln_fold_prep_kernel<<<(n_out + 7) / 8, 256, 0, st>>>((const __nv_bfloat16*)W, bias, g, beta, n_out, K,
                                                         (__nv_bfloat16*)w_out, c_out, b_out);
    return cudaGetLastError();
}

}  // namespace rs
