// Device helpers of the pipelined kernel: warp reductions through redux, order-preserving
// float/int map, packed bf16 maximum, power-of-two construction, conversion-free ceil.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bebop_common.cuh"

namespace bebop {

__device__ __forceinline__ uint32_t max_nan_bf16x2(uint32_t a, uint32_t b) {
    uint32_t r; asm("max.NaN.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b)); return r;
}
__device__ __forceinline__ int redux_max(int v) {
    int r; asm volatile("redux.sync.max.s32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v)); return r;
}
// order-preserving float <-> int map (canonical NaN sorts above +inf)
__device__ __forceinline__ int f2ord(float f) { int b = __float_as_int(f); return b ^ ((b >> 31) & 0x7fffffff); }
__device__ __forceinline__ float ord2f(int i) { return __int_as_float(i ^ ((i >> 31) & 0x7fffffff)); }

// 2^k as a double for k in [-1022, 1023], else 0 (k below) -- exact
__device__ __forceinline__ double pow2d(int k) { return k < -1022 ? 0.0 : __hiloint2double((1023 + k) << 20, 0); }
// 2^k as a float for k in [-126, 127] (0 below): exact
__device__ __forceinline__ float pow2f(int k) { return k < -126 ? 0.f : __int_as_float((127 + k) << 23); }
__device__ __forceinline__ double shfl_xor_d(double v, int m) { return __shfl_xor_sync(0xffffffffu, v, m); }
__device__ __forceinline__ double shfl_up_d(double v, int d) { return __shfl_up_sync(0xffffffffu, v, d); }

// max over the elements of one 16-byte vector, NaN-propagating
template <int DT> __device__ __forceinline__ float vec_max(const uint4& v);
template <> __device__ __forceinline__ float vec_max<0>(const uint4& v) {
    return max_nan(max_nan(__uint_as_float(v.x), __uint_as_float(v.y)),
                   max_nan(__uint_as_float(v.z), __uint_as_float(v.w)));
}
template <> __device__ __forceinline__ float vec_max<1>(const uint4& v) {
    uint32_t m = max_nan_bf16x2(max_nan_bf16x2(v.x, v.y), max_nan_bf16x2(v.z, v.w));
    return max_nan(__uint_as_float(m << 16), __uint_as_float(m & 0xffff0000u));
}
// set the lanes at or beyond `keep` to -inf (register-only: no address is taken)
template <int DT> __device__ __forceinline__ void mask_tail(uint4& v, int keep) {
    if (DT == 0) {
        if (keep <= 0) v.x = kNegInfBits;
        if (keep <= 1) v.y = kNegInfBits;
        if (keep <= 2) v.z = kNegInfBits;
        if (keep <= 3) v.w = kNegInfBits;
    } else {
        const uint32_t lo = 0x0000ff80u, hi = 0xff800000u;
        if (keep <= 0) v.x = (v.x & 0xffff0000u) | lo;
        if (keep <= 1) v.x = (v.x & 0x0000ffffu) | hi;
        if (keep <= 2) v.y = (v.y & 0xffff0000u) | lo;
        if (keep <= 3) v.y = (v.y & 0x0000ffffu) | hi;
        if (keep <= 4) v.z = (v.z & 0xffff0000u) | lo;
        if (keep <= 5) v.z = (v.z & 0x0000ffffu) | hi;
        if (keep <= 6) v.w = (v.w & 0xffff0000u) | lo;
        if (keep <= 7) v.w = (v.w & 0x0000ffffu) | hi;
    }
}



// ceil(x) for |x| < 2^22 without the conversion pipe: returns the integer and, in *r, the same value as a float
__device__ __forceinline__ int ceil_alu(float x, float* r) {
    const float magic = 12582912.f;               // 1.5 * 2^23
    float y = x + magic;                          // round to nearest integer
    int i = __float_as_int(y) - 0x4B400000;
    float f = y - magic;
    if (f < x) { f += 1.f; i += 1; }
    *r = f;
    return i;
}

}  // namespace bebop
