// Device helpers: streaming 128-bit loads, storage-type unpacking, block reductions.
#pragma once

#include "qn_internal.h"

namespace qn {

template <typename T>
struct Storage;

template <>
struct Storage<float> {
    static constexpr int kVec = 4;  // elements per 16-byte vector
    __device__ static __forceinline__ float get(const uint4& v, int e) {
        const uint32_t w = e == 0 ? v.x : e == 1 ? v.y : e == 2 ? v.z : v.w;
        return __uint_as_float(w);
    }
    __device__ static __forceinline__ float load1(const float* p) { return __ldg(p); }
    __device__ static __forceinline__ void store1(float* p, float x) { *p = x; }
    __device__ static __forceinline__ uint4 pack(const float* x) {
        return make_uint4(__float_as_uint(x[0]), __float_as_uint(x[1]), __float_as_uint(x[2]), __float_as_uint(x[3]));
    }
};

template <>
struct Storage<__nv_bfloat16> {
    static constexpr int kVec = 8;
    __device__ static __forceinline__ float get(const uint4& v, int e) {
        const uint32_t w = (e >> 1) == 0 ? v.x : (e >> 1) == 1 ? v.y : (e >> 1) == 2 ? v.z : v.w;
        return __uint_as_float((e & 1) ? (w & 0xffff0000u) : (w << 16));
    }
    __device__ static __forceinline__ float load1(const __nv_bfloat16* p) {
        return __uint_as_float(static_cast<uint32_t>(__ldg(reinterpret_cast<const unsigned short*>(p))) << 16);
    }
    __device__ static __forceinline__ void store1(__nv_bfloat16* p, float x) { *p = __float2bfloat16_rn(x); }
    __device__ static __forceinline__ uint4 pack(const float* x) {
        uint32_t w[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            // cvt.rn.bf16x2.f32 d, a, b: a -> upper half, b -> lower half
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w[i]) : "f"(x[2 * i + 1]), "f"(x[2 * i]));
        }
        return make_uint4(w[0], w[1], w[2], w[3]);
    }
};

// 16-byte read-only load that does not allocate in L1 (every input element is read once per pass).
__device__ __forceinline__ uint4 ldg_stream16(const void* p) {
    uint4 v;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
                 : "l"(p));
    return v;
}

// 32-byte read-only load (one full sector per request; the address must be 32-byte aligned).
__device__ __forceinline__ void ldg_stream32(const void* p, uint4& a, uint4& b) {
    asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                 : "=r"(a.x), "=r"(a.y), "=r"(a.z), "=r"(a.w), "=r"(b.x), "=r"(b.y), "=r"(b.z), "=r"(b.w)
                 : "l"(p));
}

// 16-byte streaming store (written once, not re-read by this kernel).
__device__ __forceinline__ void stg_stream16(void* p, const uint4& v) {
    asm volatile("st.global.cs.v4.u32 [%0], {%1,%2,%3,%4};" ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w)
                 : "memory");
}

// Sum over the warp in a fixed butterfly order; every lane ends with the same value.
__device__ __forceinline__ double warp_sum(double x) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) x += __shfl_xor_sync(0xffffffffu, x, o);
    return x;
}


// ---- mbarrier helpers (shared memory barriers that track arrivals and bytes of bulk copies) -------------
constexpr uint32_t kWaitLimit = 1u << 24;         // polls per wait before giving up, whatever the clock says
constexpr uint64_t kWaitLimitNs = 1000000000ull;  // and one second by the global timer, checked every 256 polls

__device__ __forceinline__ uint64_t global_timer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint64_t* bar, uint32_t parity) {
    uint32_t done;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(done)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return done != 0;
}
// Bounded wait.  Returns false (and raises the abort flag) when the limit runs out or another thread
// of the CTA has already given up.
template <bool kBackOff = true>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, volatile int* abort) {
    if (mbar_try(bar, parity)) return true;  // the common case costs one shared-memory round trip
    if (*abort) return false;
    const uint64_t t0 = global_timer_ns();
    for (uint32_t it = 0; it < kWaitLimit; ++it) {
        if (mbar_try(bar, parity)) return true;
        // waiting warps sleep between polls so that they do not take issue slots from the others (a warp on the
        // critical path polls without sleeping)
        if (kBackOff) __nanosleep(64);
        if ((it & 255u) == 255u) {
            if (*abort) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) break;
        }
    }
    *abort = 1;
    return false;
}

// Arrive and announce `bytes` of bulk-copy traffic that will complete on this barrier.
__device__ __forceinline__ void mbar_arrive_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
// Bulk copy global -> shared (TMA, untiled): 16-byte aligned addresses, size a multiple of 16 bytes; the bytes
// complete on `bar`.
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(smem_dst)),
                 "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}
// Bulk copy shared -> global as one bulk group; bulk_store_wait_read returns once the copies issued by this
// thread have read their shared memory (which may then be overwritten).
__device__ __forceinline__ void bulk_store(void* gdst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst), "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_store_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_store_wait_read() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_store_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }

}  // namespace qn
