// Device helpers shared by the SparQ kernels (sm_100a).
#pragma once
#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <math_constants.h>
#include <stdint.h>

#include "sparq.h"

namespace sparq {

constexpr int D = SPARQ_HEAD_DIM;        // head dimension d_h
constexpr unsigned FULL = 0xffffffffu;
constexpr float LOG2E = 1.4426950408889634f;

__device__ __forceinline__ void raise_status(int32_t* status, int code) {
    if (status) atomicMax(status, code);
}

// ---- fp16 -> fp64 without the slow 64-bit conversion pipe -------------------------------
// The 15 exponent+mantissa bits of a binary16 value, placed at bits 24..10 of the high word
// of a binary64, give exactly value * 2^-1008 (subnormals included: they land on binary64
// subnormals with the same scaling; an all-ones exponent maps to a finite value, so no bit
// pattern can produce an infinity or a NaN).  The query side carries the factor 2^+1008, so
// every product q_j * K[t, j] is formed exactly and the fp64 FMA chain equals the plain
// fp64 sum taken in the same order.
__device__ __forceinline__ double h2d_lo(uint32_t w) {   // low half of a packed half2
    return __hiloint2double((int)(((w & 0x8000u) << 16) | ((w & 0x7fffu) << 10)), 0);
}
__device__ __forceinline__ double h2d_hi(uint32_t w) {   // high half of a packed half2
    return __hiloint2double((int)((w & 0x80000000u) | ((w >> 6) & 0x01fffc00u)), 0);
}
__device__ __forceinline__ double h2d_scalar(uint16_t h) { return h2d_lo((uint32_t)h); }

// order-preserving integer keys (larger value <-> larger key); -0 is folded into +0 first
__device__ __forceinline__ uint32_t key32(float f) {
    uint32_t b = __float_as_uint(f + 0.0f);
    return b ^ ((uint32_t)((int32_t)b >> 31) | 0x80000000u);
}
__device__ __forceinline__ float unkey32(uint32_t u) {
    return __uint_as_float((u & 0x80000000u) ? (u ^ 0x80000000u) : ~u);
}
__device__ __forceinline__ unsigned long long key64(double f) {
    unsigned long long b = (unsigned long long)__double_as_longlong(f + 0.0);
    return b ^ ((unsigned long long)((long long)b >> 63) | 0x8000000000000000ull);
}

__device__ __forceinline__ uint4 ld_stream(const uint4* p) {   // read-once data: keep it out of L1
    uint4 v;
    asm("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
        : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
    return v;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(FULL, v, o);
    return v;
}

// ---- mbarrier + bulk asynchronous copy (global -> shared, completion on an mbarrier) -----
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_init_fence() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// The same poll, but the hardware may park the thread for up to `ns` nanoseconds before it answers,
// so a waiting warp does not eat issue slots.
__device__ __forceinline__ bool mbar_try_wait_parked(uint64_t* bar, uint32_t parity, uint32_t ns) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity), "r"(ns) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after `limit` polls and returns false (the caller reports an error
// status and leaves; it never spins forever).
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, int limit) {
    for (int i = 0; i < limit; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return false;
}
// src and dst 16-byte aligned, bytes a multiple of 16.  No multicast.
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

}  // namespace sparq
