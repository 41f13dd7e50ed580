// fp32-FMA contraction path: a tiled GEMM with the block's epilogues and a
// streaming-softmax attention that keeps one query row per thread.  It serves
// the RS_F32 storage type (tensor cores have no fp32 x fp32 mode with fp32
// products) and is the on-device cross-check for the tcgen05 kernels.
#include <math.h>

#include "rs_internal.h"
#include "rs_device.cuh"

namespace rs {

namespace {

// ---------------------------------------------------------------- GEMM
// out[M, N] = act(A[M, K] . W[N, K]^T + bias) + residual, 64x64 tile per CTA,
// 16x16 threads each owning a 4x4 micro-tile, K in slabs of 16.
constexpr int TM = 64, TN = 64, TK = 16;

__device__ __forceinline__ float load_any(const void* p, long long i, int dtype) {
    return dtype == RS_BF16 ? __bfloat162float(((const __nv_bfloat16*)p)[i]) : ((const float*)p)[i];
}
__device__ __forceinline__ void store_any(void* p, long long i, int dtype, float v) {
    if (dtype == RS_BF16) ((__nv_bfloat16*)p)[i] = __float2bfloat16_rn(v);
    else ((float*)p)[i] = v;
}

template <typename T>
__global__ void __launch_bounds__(256)
gemm_simt_kernel(const T* __restrict__ A, const T* __restrict__ W, const float* __restrict__ bias,
                 int gelu, const void* __restrict__ residual, int res_dtype, void* __restrict__ out,
                 int out_dtype, long long M, int N, int K) {
    __shared__ float As[TK][TM + 1];
    __shared__ float Ws[TK][TN + 1];
    const int tx = threadIdx.x & 15, ty = threadIdx.x >> 4;
    const long long m0 = (long long)blockIdx.y * TM;
    const int n0 = blockIdx.x * TN;
    float acc[4][4] = {};
    for (int k0 = 0; k0 < K; k0 += TK) {
        for (int e = threadIdx.x; e < TM * TK; e += 256) {
            const int r = e / TK, c = e % TK;
            const long long gm = m0 + r;
            As[c][r] = (gm < M && k0 + c < K) ? to_float(A[gm * K + k0 + c]) : 0.f;
            const int gn = n0 + r;
            Ws[c][r] = (gn < N && k0 + c < K) ? to_float(W[(long long)gn * K + k0 + c]) : 0.f;
        }
        __syncthreads();
#pragma unroll
        for (int c = 0; c < TK; ++c) {
            float a[4], w[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) { a[i] = As[c][ty * 4 + i]; w[i] = Ws[c][tx * 4 + i]; }
#pragma unroll
            for (int i = 0; i < 4; ++i)
#pragma unroll
                for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const long long gm = m0 + ty * 4 + i;
        if (gm >= M) continue;
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int gn = n0 + tx * 4 + j;
            if (gn >= N) continue;
            float v = acc[i][j] + (bias ? bias[gn] : 0.f);
            if (gelu) v = 0.5f * v * (1.f + erff(v * 0.70710678118654752f));
            if (residual) v += load_any(residual, gm * N + gn, res_dtype);
            store_any(out, gm * N + gn, out_dtype, v);
        }
    }
}

// ---------------------------------------------------------------- attention
// Eq. sa with a running max / running sum (no N x N buffer): one thread per
// query row, keys and values of one head staged through shared memory 32 rows
// at a time, head dimension 64.
constexpr int ADH = 64, AQ = 128, AKV = 32;

template <typename T>
__global__ void __launch_bounds__(AQ)
attn_simt_kernel(const T* __restrict__ q, const T* __restrict__ k, const T* __restrict__ v,
                 T* __restrict__ out, int N, int H, float scale, long long qb, long long qr,
                 long long qh, long long kb, long long kr, long long kh, long long vb, long long vr,
                 long long vh) {
    __shared__ float Ks[AKV][ADH];
    __shared__ float Vs[AKV][ADH];
    const int b = blockIdx.z, h = blockIdx.y;
    const int i = blockIdx.x * AQ + threadIdx.x;
    const bool active = i < N;
    float qreg[ADH], o[ADH];
    const T* qp = q + b * qb + (long long)(active ? i : 0) * qr + h * qh;
#pragma unroll
    for (int c = 0; c < ADH; ++c) { qreg[c] = to_float(qp[c]) * scale; o[c] = 0.f; }
    float mrun = -INFINITY, lrun = 0.f;
    for (int j0 = 0; j0 < N; j0 += AKV) {
        __syncthreads();
        for (int e = threadIdx.x; e < AKV * ADH; e += AQ) {
            const int r = e / ADH, c = e % ADH;
            const int j = j0 + r;
            Ks[r][c] = j < N ? to_float(k[b * kb + (long long)j * kr + h * kh + c]) : 0.f;
            Vs[r][c] = j < N ? to_float(v[b * vb + (long long)j * vr + h * vh + c]) : 0.f;
        }
        __syncthreads();
        float s[AKV];
        float mx = mrun;
#pragma unroll
        for (int r = 0; r < AKV; ++r) {
            float acc = 0.f;
#pragma unroll
            for (int c = 0; c < ADH; ++c) acc = fmaf(qreg[c], Ks[r][c], acc);
            s[r] = (j0 + r < N) ? acc : -INFINITY;
            mx = fmaxf(mx, s[r]);
        }
        const float corr = expf(mrun - mx);      // exp(-inf) = 0 on the first tile
        lrun *= corr;
#pragma unroll
        for (int c = 0; c < ADH; ++c) o[c] *= corr;
#pragma unroll
        for (int r = 0; r < AKV; ++r) {
            const float p = expf(s[r] - mx);
            lrun += p;
#pragma unroll
            for (int c = 0; c < ADH; ++c) o[c] = fmaf(p, Vs[r][c], o[c]);
        }
        mrun = mx;
    }
    if (active) {
        const float inv = 1.f / lrun;
        T* op = out + ((long long)b * N + i) * ((long long)H * ADH) + h * ADH;
#pragma unroll
        for (int c = 0; c < ADH; ++c) op[c] = from_float<T>(o[c] * inv);
    }
}

}  // namespace

cudaError_t launch_gemm_simt(rs_dtype in_dtype, const void* A, const void* W, const float* bias,
                             int gelu, const void* residual, rs_dtype res_dtype, void* out,
                             rs_dtype out_dtype, long long M, int N, int K, cudaStream_t st) {
    if (M == 0 || N == 0) return cudaSuccess;
    const dim3 grid((N + TN - 1) / TN, (unsigned)((M + TM - 1) / TM));
    if (in_dtype == RS_BF16)
        gemm_simt_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)A, (const __nv_bfloat16*)W, bias,
                                                             gelu, residual, res_dtype, out, out_dtype, M, N, K);
    else
        gemm_simt_kernel<float><<<grid, 256, 0, st>>>((const float*)A, (const float*)W, bias, gelu, residual,
                                                     res_dtype, out, out_dtype, M, N, K);
    return cudaGetLastError();
}

cudaError_t launch_attn_simt(const rs_attn_desc& d, const void* q, const void* k, const void* v,
                             void* out, cudaStream_t st) {
    if (d.B == 0 || d.N == 0) return cudaSuccess;
    const float scale = d.scale != 0.f ? d.scale : 1.f / sqrtf((float)d.head_dim);
    const dim3 grid((d.N + AQ - 1) / AQ, d.H, d.B);
    if (d.dtype == RS_BF16)
        attn_simt_kernel<__nv_bfloat16><<<grid, AQ, 0, st>>>(
            (const __nv_bfloat16*)q, (const __nv_bfloat16*)k, (const __nv_bfloat16*)v, (__nv_bfloat16*)out, d.N, d.H,
            scale, d.q_batch_stride, d.q_row_stride, d.q_head_stride, d.k_batch_stride, d.k_row_stride,
            d.k_head_stride, d.v_batch_stride, d.v_row_stride, d.v_head_stride);
    else
        attn_simt_kernel<float><<<grid, AQ, 0, st>>>(
            (const float*)q, (const float*)k, (const float*)v, (float*)out, d.N, d.H, scale, d.q_batch_stride,
            d.q_row_stride, d.q_head_stride, d.k_batch_stride, d.k_row_stride, d.k_head_stride,
            d.v_batch_stride, d.v_row_stride, d.v_head_stride);
    return cudaGetLastError();
}

}  // namespace rs
