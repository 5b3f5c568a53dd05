// Shared device helpers of the verify kernels: element traits, 128-bit loads,
// NaN-propagating max, online-softmax merges, warp/block reductions.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace bebop {

constexpr int ST_NONFINITE = 1, ST_EMPTY = 2, ST_BAD_TOKEN = 4, ST_ZERO_RESID = 8, ST_BAD_TEMP = 16,
              ST_WAIT = 32;
constexpr int ST_FATAL = ST_NONFINITE | ST_EMPTY | ST_BAD_TOKEN | ST_BAD_TEMP;
constexpr float kLog2e = 1.4426950408889634f;
constexpr uint32_t kNegInfBits = 0xff800000u;

// DT = 0: fp32 logits (4 per 16-byte vector); DT = 1: bf16 logits (8 per vector).
template <int DT> struct Elem;
template <> struct Elem<0> { static constexpr int VEC = 4; static constexpr int BYTES = 4; };
template <> struct Elem<1> { static constexpr int VEC = 8; static constexpr int BYTES = 2; };

__device__ __forceinline__ uint4 ldg16_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}
__device__ __forceinline__ uint4 ldg16(const void* p) { return *reinterpret_cast<const uint4*>(p); }

__device__ __forceinline__ float ex2f(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// max that returns NaN if either operand is NaN
__device__ __forceinline__ float max_nan(float a, float b) {
    float r;
    asm("max.NaN.f32 %0, %1, %2;" : "=f"(r) : "f"(a), "f"(b));
    return r;
}

template <int DT> __device__ __forceinline__ void unpack(const uint4& v, float* f);
template <> __device__ __forceinline__ void unpack<0>(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x); f[1] = __uint_as_float(v.y);
    f[2] = __uint_as_float(v.z); f[3] = __uint_as_float(v.w);
}
template <> __device__ __forceinline__ void unpack<1>(const uint4& v, float* f) {
    f[0] = __uint_as_float(v.x << 16); f[1] = __uint_as_float(v.x & 0xffff0000u);
    f[2] = __uint_as_float(v.y << 16); f[3] = __uint_as_float(v.y & 0xffff0000u);
    f[4] = __uint_as_float(v.z << 16); f[5] = __uint_as_float(v.z & 0xffff0000u);
    f[6] = __uint_as_float(v.w << 16); f[7] = __uint_as_float(v.w & 0xffff0000u);
}

// A 16-byte vector of -inf logits (used for out-of-range loads).
template <int DT> __device__ __forceinline__ uint4 neg_inf_vec() {
    if (DT == 0) return make_uint4(kNegInfBits, kNegInfBits, kNegInfBits, kNegInfBits);
    return make_uint4(0xff80ff80u, 0xff80ff80u, 0xff80ff80u, 0xff80ff80u);
}

// Load vector `iv` of a row and unpack it; lanes at or beyond V become -inf.
template <int DT>
__device__ __forceinline__ void load_vec(const char* row, int64_t iv, int V, float* f) {
    constexpr int VEC = Elem<DT>::VEC;
    uint4 v = ldg16_stream(row + iv * 16);
    unpack<DT>(v, f);
    int base = (int)(iv * VEC);
    if (base + VEC > V) {
#pragma unroll
        for (int j = 0; j < VEC; ++j) if (base + j >= V) f[j] = __uint_as_float(kNegInfBits);
    }
}

// Read one logit of a row as float.
template <int DT> __device__ __forceinline__ float load_one(const char* row, int64_t v) {
    if (DT == 0) return reinterpret_cast<const float*>(row)[v];
    uint32_t h = reinterpret_cast<const unsigned short*>(row)[v];
    return __uint_as_float(h << 16);
}

// (m, S) of an online softmax: S = sum exp2((x - m) * c).  Merge keeps NaN and
// treats m = -inf as the empty partial.
struct MS { float m, s; };
__device__ __forceinline__ MS ms_merge(MS a, MS b, float c) {
    MS r;
    r.m = max_nan(a.m, b.m);
    if (r.m == __uint_as_float(kNegInfBits)) { r.s = 0.f; return r; }
    r.s = a.s * ex2f((a.m - r.m) * c) + b.s * ex2f((b.m - r.m) * c);
    return r;
}
__device__ __forceinline__ MS ms_warp(MS v, float c) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
        MS w;
        w.m = __shfl_xor_sync(0xffffffffu, v.m, o);
        w.s = __shfl_xor_sync(0xffffffffu, v.s, o);
        v = ms_merge(v, w, c);
    }
    return v;
}

struct MSd { double m, s; };
__device__ __forceinline__ MSd msd_merge(MSd a, MSd b) {
    MSd r;
    r.m = (a.m != a.m || b.m != b.m) ? (a.m + b.m) : fmax(a.m, b.m);
    if (r.m == -INFINITY) { r.s = 0.0; return r; }
    r.s = a.s * exp(a.m - r.m) + b.s * exp(b.m - r.m);
    return r;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Slice [begin, end) of the row's 16-byte vectors owned by split `s` of `nsplit`.
__device__ __forceinline__ void slice_range(int nvec, int nsplit, int s, int& begin, int& end) {
    int per = (nvec + nsplit - 1) / nsplit;
    begin = min(s * per, nvec);
    end = min(begin + per, nvec);
}

}  // namespace bebop
