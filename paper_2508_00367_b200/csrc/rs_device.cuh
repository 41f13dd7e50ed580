// Small device helpers: typed 16-byte loads/stores and warp reductions.
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>

namespace rs {

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute
// may start while its predecessor in the stream is still draining.  grid_dep_launch() lets the
// successor be scheduled early; grid_dep_wait() blocks until the predecessor has completed and
// its writes are visible, and must come before the first access to global memory.  Both are
// no-ops for a kernel launched the ordinary way.
__device__ __forceinline__ void grid_dep_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void grid_dep_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// 16-byte read of data that is used once: read-only path, no L1 allocation.
__device__ __forceinline__ uint4 ld_stream(const uint4* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}
__device__ __forceinline__ float4 ld_stream(const float4* p) {
    const uint4 v = ld_stream(reinterpret_cast<const uint4*>(p));
    return make_float4(__uint_as_float(v.x), __uint_as_float(v.y), __uint_as_float(v.z), __uint_as_float(v.w));
}

template <typename T> struct Vec16;           // one 16-byte vector of T
template <> struct Vec16<float> {
    static constexpr int N = 4;
    float v[4];
    __device__ __forceinline__ void load(const float* p) {
        float4 t = ld_stream(reinterpret_cast<const float4*>(p));
        v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    }
    __device__ __forceinline__ void store(float* p) const {
        *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    }
};
template <> struct Vec16<__nv_bfloat16> {
    static constexpr int N = 8;
    float v[8];
    __device__ __forceinline__ void load(const __nv_bfloat16* p) {
        uint4 t = ld_stream(reinterpret_cast<const uint4*>(p));
        const uint32_t w[4] = {t.x, t.y, t.z, t.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            v[2 * i] = __uint_as_float(w[i] << 16);
            v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
    __device__ __forceinline__ void store(__nv_bfloat16* p) const {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t*>(&h);
        }
        *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
    }
};

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    return v;
}

template <typename TO, int N>
__device__ __forceinline__ void store_n(TO* p, const float* v);
template <> __device__ __forceinline__ void store_n<float, 4>(float* p, const float* v) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
}
template <> __device__ __forceinline__ void store_n<float, 8>(float* p, const float* v) {
    *reinterpret_cast<float4*>(p) = make_float4(v[0], v[1], v[2], v[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(v[4], v[5], v[6], v[7]);
}
template <> __device__ __forceinline__ void store_n<__nv_bfloat16, 4>(__nv_bfloat16* p, const float* v) {
    __nv_bfloat162 a = __floats2bfloat162_rn(v[0], v[1]);
    __nv_bfloat162 b = __floats2bfloat162_rn(v[2], v[3]);
    *reinterpret_cast<uint2*>(p) = make_uint2(*reinterpret_cast<uint32_t*>(&a), *reinterpret_cast<uint32_t*>(&b));
}
template <> __device__ __forceinline__ void store_n<__nv_bfloat16, 8>(__nv_bfloat16* p, const float* v) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        __nv_bfloat162 h = __floats2bfloat162_rn(v[2 * i], v[2 * i + 1]);
        w[i] = *reinterpret_cast<uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
}

// 16 bytes of T as floats.
template <typename T> __device__ __forceinline__ void unpack16(const uint4& r, float (&v)[Vec16<T>::N]);
template <> __device__ __forceinline__ void unpack16<float>(const uint4& r, float (&v)[4]) {
    v[0] = __uint_as_float(r.x); v[1] = __uint_as_float(r.y); v[2] = __uint_as_float(r.z); v[3] = __uint_as_float(r.w);
}
template <> __device__ __forceinline__ void unpack16<__nv_bfloat16>(const uint4& r, float (&v)[8]) {
    const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        v[2 * i] = __uint_as_float(w[i] << 16);
        v[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

// LayerNorm of one token row held by a warp as packed 16-byte pieces: lane l owns pieces
// l, l + 32, ... (nvec = D / Vec16<TI>::N of them, at most 32 * MAXV).  Mean, then the biased
// variance about it, then the affine map; the row is unpacked once per pass, which keeps the
// callers near 48 to 64 registers.  Every kernel that normalises a row calls this, so a row has
// the same result whichever kernel produced it.
template <typename TI, typename TO, int MAXV>
__device__ __forceinline__ void layernorm_row(const uint4 (&raw)[MAXV], int nvec, int lane,
                                              const float* __restrict__ gamma, const float* __restrict__ beta,
                                              float eps, int D, TO* __restrict__ orow) {
    constexpr int VN = Vec16<TI>::N;
    float sum = 0.f;
#pragma unroll
    for (int j = 0; j < MAXV; ++j) {
        if (j * 32 + lane < nvec) {
            float v[VN];
            unpack16<TI>(raw[j], v);
#pragma unroll
            for (int e = 0; e < VN; ++e) sum += v[e];
        }
    }
    const float mu = warp_sum(sum) / (float)D;
    float sq = 0.f;
#pragma unroll
    for (int j = 0; j < MAXV; ++j) {
        if (j * 32 + lane < nvec) {
            float v[VN];
            unpack16<TI>(raw[j], v);
#pragma unroll
            for (int e = 0; e < VN; ++e) { const float dd = v[e] - mu; sq += dd * dd; }
        }
    }
    const float rstd = rsqrtf(warp_sum(sq) / (float)D + eps);
#pragma unroll
    for (int j = 0; j < MAXV; ++j) {
        const int iv = j * 32 + lane;
        if (iv < nvec) {
            float v[VN], y[VN];
            unpack16<TI>(raw[j], v);
#pragma unroll
            for (int e = 0; e < VN; e += 4) {
                const float4 g = __ldg(reinterpret_cast<const float4*>(gamma + iv * VN + e));
                const float4 bt = __ldg(reinterpret_cast<const float4*>(beta + iv * VN + e));
                y[e + 0] = (v[e + 0] - mu) * rstd * g.x + bt.x;
                y[e + 1] = (v[e + 1] - mu) * rstd * g.y + bt.y;
                y[e + 2] = (v[e + 2] - mu) * rstd * g.z + bt.z;
                y[e + 3] = (v[e + 3] - mu) * rstd * g.w + bt.w;
            }
            store_n<TO, VN>(orow + iv * VN, y);
        }
    }
}

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_float(float v);
template <> __device__ __forceinline__ float from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float v) {
    return __float2bfloat16_rn(v);
}

}  // namespace rs
