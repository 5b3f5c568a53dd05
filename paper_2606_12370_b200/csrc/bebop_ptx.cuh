// PTX helpers of the cluster kernels: cluster identity and barriers, distributed
// shared memory, mbarriers (local and remote), bulk asynchronous copies, packed
// bf16 max, warp reductions, tensor-memory loads and stores.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

#include "bebop_common.cuh"

namespace bebop {

constexpr uint32_t kWaitPolls = 1u << 20;   // bound of every spin on an mbarrier

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t r; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t cluster_id() { uint32_t r; asm volatile("mov.u32 %0, %%clusterid.x;" : "=r"(r)); return r; }
__device__ __forceinline__ uint32_t num_clusters() { uint32_t r; asm volatile("mov.u32 %0, %%nclusterid.x;" : "=r"(r)); return r; }
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ uint32_t mapa(uint32_t addr, uint32_t rank) {
    uint32_t r; asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank)); return r;
}
__device__ __forceinline__ void st_cluster_v4(uint32_t addr, uint4 v) {
    asm volatile("st.shared::cluster.v4.b32 [%0], {%1,%2,%3,%4};" :: "r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" :: "r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait; returns false if it gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitPolls; ++i) if (mbar_try_wait(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 :: "r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
// arrive on an mbarrier of another CTA of the cluster (address from mapa), release at cluster scope
__device__ __forceinline__ void mbar_arrive_remote(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" :: "r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait with cluster-scope acquire; returns false if it gave up.
__device__ __forceinline__ bool mbar_wait_cluster(uint32_t bar, uint32_t parity) {
    for (uint32_t i = 0; i < kWaitPolls; ++i) if (mbar_try_wait_cluster(bar, parity)) return true;
    return false;
}
__device__ __forceinline__ void st_cluster_v2(uint32_t addr, uint32_t x, uint32_t y) {
    asm volatile("st.shared::cluster.v2.b32 [%0], {%1,%2};" :: "r"(addr), "r"(x), "r"(y) : "memory");
}
__device__ __forceinline__ void st_cluster_b32(uint32_t addr, uint32_t x) {
    asm volatile("st.shared::cluster.b32 [%0], %1;" :: "r"(addr), "r"(x) : "memory");
}
__device__ __forceinline__ uint32_t redux_add(uint32_t v) {
    uint32_t r; asm volatile("redux.sync.add.u32 %0, %1, 0xffffffff;" : "=r"(r) : "r"(v)); return r;
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
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



// ----------------------------------------------------------------- tensor memory
// One warp allocates / frees all 512 columns of the SM's tensor memory.
__device__ __forceinline__ void tmem_alloc512(uint32_t smem_result_addr) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_result_addr), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc512(uint32_t taddr) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(taddr), "r"(512u) : "memory");
}
__device__ __forceinline__ void tmem_fence_before_sync() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tmem_fence_after_sync() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
// Each lane stores / loads 8 consecutive 32-bit columns of its own tensor-memory lane.
__device__ __forceinline__ void tmem_st8(uint32_t taddr, const float* v) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};"
                 :: "r"(taddr), "f"(v[0]), "f"(v[1]), "f"(v[2]), "f"(v[3]), "f"(v[4]), "f"(v[5]), "f"(v[6]), "f"(v[7]) : "memory");
}
__device__ __forceinline__ void tmem_ld8(uint32_t taddr, float* v) {
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=f"(v[0]), "=f"(v[1]), "=f"(v[2]), "=f"(v[3]), "=f"(v[4]), "=f"(v[5]), "=f"(v[6]), "=f"(v[7]) : "r"(taddr) : "memory");
}
__device__ __forceinline__ void tmem_wait_st() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
__device__ __forceinline__ void tmem_wait_ld() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// 2^k as a float for k in [-126, 127] (0 below): exact
__device__ __forceinline__ float pow2f(int k) { return k < -126 ? 0.f : __int_as_float((127 + k) << 23); }

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
