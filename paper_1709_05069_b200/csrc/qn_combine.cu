// Final streaming pass: theta_new = thetabar - tau*(gbar - G d + Theta d)  (paper, Eq. (2) with the
// operator of Eq. (4) applied to gbar; G d and Theta d are the two sums of Eq. (4) collapsed onto the
// m-vector d built by the solve kernel).  With c = tau*(d - mean(d)), sum(c) = 0 and
//     theta_new[i] = mean_k theta[k][i] - tau * mean_k g[k][i]
//                    + sum_k c[k] * ((g[k][i] - g[0][i]) - (theta[k][i] - theta[0][i])).
// Differences against Worker 0 are formed before the multiplication so that the rounding of each
// term is relative to the Workers' spread, not to the magnitude of theta and g.  fp32 arithmetic,
// fixed summation order k = 0..m-1, one rounding to the storage type.  Neither the means nor the
// centred matrices are ever stored: the pass reads 2*m*n elements and writes n.
#include "qn_device.cuh"

namespace qn {

constexpr int kCombineThreads = 256;
constexpr int kCombineUnroll = 4;  // Workers whose loads are in flight together

template <typename T, bool kAligned>
__global__ void __launch_bounds__(kCombineThreads)
combine_kernel(const T* __restrict__ theta, const T* __restrict__ g, int64_t n, int m,
               const qn_coef_block* __restrict__ coef, T* __restrict__ out, const T* __restrict__ base) {
    constexpr int kCols = kAligned ? Storage<T>::kVec : 1;
    __shared__ float c_sh[QN_MAX_M];
    if (threadIdx.x < QN_MAX_M) c_sh[threadIdx.x] = coef->c[threadIdx.x];
    const float tau = coef->tau, inv_m = coef->inv_m;
    __syncthreads();

    const int64_t nitems = kAligned ? n / kCols : n;
    for (int64_t item = (int64_t)blockIdx.x * kCombineThreads + threadIdx.x; item < nitems;
         item += (int64_t)gridDim.x * kCombineThreads) {
        const int64_t i0 = item * kCols;
        float th0[kCols], g0[kCols], sth[kCols], sg[kCols], acc[kCols];
        {
            uint4 a, b;
            if (kAligned) {
                a = ldg_stream16(theta + i0);
                b = ldg_stream16(g + i0);
            } else {
                a.x = __float_as_uint(Storage<T>::load1(theta + i0));
                b.x = __float_as_uint(Storage<T>::load1(g + i0));
            }
#pragma unroll
            for (int e = 0; e < kCols; ++e) {
                th0[e] = kAligned ? Storage<T>::get(a, e) : __uint_as_float(a.x);
                g0[e] = kAligned ? Storage<T>::get(b, e) : __uint_as_float(b.x);
                sth[e] = th0[e];
                sg[e] = g0[e];
                acc[e] = 0.f;
            }
        }
        int k = 1;
        for (; k + kCombineUnroll <= m; k += kCombineUnroll) {
            uint4 a[kCombineUnroll], b[kCombineUnroll];
#pragma unroll
            for (int u = 0; u < kCombineUnroll; ++u) {
                if (kAligned) {
                    a[u] = ldg_stream16(theta + (int64_t)(k + u) * n + i0);
                    b[u] = ldg_stream16(g + (int64_t)(k + u) * n + i0);
                } else {
                    a[u].x = __float_as_uint(Storage<T>::load1(theta + (int64_t)(k + u) * n + i0));
                    b[u].x = __float_as_uint(Storage<T>::load1(g + (int64_t)(k + u) * n + i0));
                }
            }
#pragma unroll
            for (int u = 0; u < kCombineUnroll; ++u) {
                const float ck = c_sh[k + u];
#pragma unroll
                for (int e = 0; e < kCols; ++e) {
                    const float t = kAligned ? Storage<T>::get(a[u], e) : __uint_as_float(a[u].x);
                    const float gg = kAligned ? Storage<T>::get(b[u], e) : __uint_as_float(b[u].x);
                    sth[e] += t;
                    sg[e] += gg;
                    acc[e] = fmaf(ck, (gg - g0[e]) - (t - th0[e]), acc[e]);
                }
            }
        }
        for (; k < m; ++k) {
            uint4 a, b;
            if (kAligned) {
                a = ldg_stream16(theta + (int64_t)k * n + i0);
                b = ldg_stream16(g + (int64_t)k * n + i0);
            } else {
                a.x = __float_as_uint(Storage<T>::load1(theta + (int64_t)k * n + i0));
                b.x = __float_as_uint(Storage<T>::load1(g + (int64_t)k * n + i0));
            }
            const float ck = c_sh[k];
#pragma unroll
            for (int e = 0; e < kCols; ++e) {
                const float t = kAligned ? Storage<T>::get(a, e) : __uint_as_float(a.x);
                const float gg = kAligned ? Storage<T>::get(b, e) : __uint_as_float(b.x);
                sth[e] += t;
                sg[e] += gg;
                acc[e] = fmaf(ck, (gg - g0[e]) - (t - th0[e]), acc[e]);
            }
        }
        float res[kCols];
#pragma unroll
        for (int e = 0; e < kCols; ++e) res[e] = fmaf(-tau * inv_m, sg[e], fmaf(sth[e], inv_m, acc[e]));
        if (base) {  // Eq. (4) applied to z: the correction is added to z instead of to the means
            uint4 zv;
            if (kAligned)
                zv = ldg_stream16(base + i0);
            else
                zv.x = __float_as_uint(Storage<T>::load1(base + i0));
#pragma unroll
            for (int e = 0; e < kCols; ++e) res[e] = (kAligned ? Storage<T>::get(zv, e) : __uint_as_float(zv.x)) + acc[e];
        }
        if (kAligned) {
            stg_stream16(out + i0, Storage<T>::pack(res));
        } else {
            Storage<T>::store1(out + i0, res[0]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Vector path (rows on 16-byte boundaries): the same arithmetic on pairs of columns with the packed
// fp32x2 instructions of sm_100 (add/sub/fma on two floats at once), which halves the ALU work per byte;
// with bf16 storage the scalar form spends about 70 % of the FMA-pipe slots at HBM speed.  Workers are
// processed four at a time with all eight loads in flight, the last batch predicated.
// ------------------------------------------------------------------------------------------------
typedef unsigned long long f32x2;  // two floats in one 64-bit register

__device__ __forceinline__ f32x2 pk(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpk(f32x2 v, float& lo, float& hi) { asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v)); }
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

// One work item = kPairs pairs of columns of every row: a 16-byte vector for fp32 storage (4 columns), HALF a vector for
// bf16 storage (8 bytes, 4 columns).  With whole bf16 vectors the per-thread state (five packed quantities per pair and
// the loads in flight) takes 108 registers, two CTAs of 256 fit an SM and the pass is latency-bound at 5.8 TB/s.  With
// half vectors, four Workers (eight loads) in flight and CTAs of 128 threads it takes 56 registers and nine CTAs fit:
// measured 6.5 TB/s at m = 8, 6.7 at m = 16, 7.0 at m = 64 (eight Workers in flight, 78 registers, CTAs of 256: 6.1,
// 6.5, 6.9; two Workers in flight: 5.3, 5.6, 6.0).  fp32 storage: 6.95 TB/s at m = 32 either way.
template <typename T>
struct CombineItem {
    static constexpr int kPairs = 2;
    static constexpr int kCols = 4;
    static constexpr int kThreads = sizeof(T) == 2 ? 128 : kCombineThreads;
    static constexpr int kUnroll = 4;  // Workers whose loads are in flight together
    // pair p (0 or 1) of the item as two floats
    static __device__ __forceinline__ f32x2 pair(const uint2& lo, const uint2& hi, int p);
};
template <>
__device__ __forceinline__ f32x2 CombineItem<float>::pair(const uint2& lo, const uint2& hi, int p) {
    return p == 0 ? pk(__uint_as_float(lo.x), __uint_as_float(lo.y)) : pk(__uint_as_float(hi.x), __uint_as_float(hi.y));
}
template <>
__device__ __forceinline__ f32x2 CombineItem<__nv_bfloat16>::pair(const uint2& lo, const uint2&, int p) {
    const uint32_t w = p == 0 ? lo.x : lo.y;
    return pk(__uint_as_float(w << 16), __uint_as_float(w & 0xffff0000u));
}
// the item's bytes: 16 (fp32: lo and hi) or 8 (bf16: lo only)
template <typename T>
__device__ __forceinline__ void load_item(const T* p, uint2& lo, uint2& hi) {
    if (sizeof(T) == 4) {
        asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(lo.x), "=r"(lo.y), "=r"(hi.x), "=r"(hi.y) : "l"(p));
    } else {
        asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(lo.x), "=r"(lo.y) : "l"(p));
        hi = make_uint2(0, 0);
    }
}

template <typename T>
__global__ void __launch_bounds__(CombineItem<T>::kThreads)
combine_vec_kernel(const T* __restrict__ theta, const T* __restrict__ g, int64_t n, int m,
                   const qn_coef_block* __restrict__ coef, T* __restrict__ out, const T* __restrict__ base) {
    using Item = CombineItem<T>;
    constexpr int kCols = Item::kCols, kPairs = Item::kPairs, kUnroll = Item::kUnroll, kThreads = Item::kThreads;
    __shared__ float c_sh[QN_MAX_M];
    for (int k = threadIdx.x; k < QN_MAX_M; k += kThreads) c_sh[k] = coef->c[k];
    const float tau = coef->tau, inv_m = coef->inv_m;
    __syncthreads();
    const int64_t nitems = n / kCols;
    for (int64_t item = (int64_t)blockIdx.x * kThreads + threadIdx.x; item < nitems; item += (int64_t)gridDim.x * kThreads) {
        const int64_t i0 = item * kCols;
        f32x2 th0[kPairs], g0[kPairs], sth[kPairs], sg[kPairs], acc[kPairs];
        {
            uint2 al, ah, bl, bh;
            load_item(theta + i0, al, ah);
            load_item(g + i0, bl, bh);
#pragma unroll
            for (int p = 0; p < kPairs; ++p) {
                th0[p] = sth[p] = Item::pair(al, ah, p);
                g0[p] = sg[p] = Item::pair(bl, bh, p);
                acc[p] = pk(0.f, 0.f);
            }
        }
        for (int k = 1; k < m; k += kUnroll) {
            uint2 al[kUnroll], ah[kUnroll], bl[kUnroll], bh[kUnroll];
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                if (k + u < m) {
                    load_item(theta + (int64_t)(k + u) * n + i0, al[u], ah[u]);
                    load_item(g + (int64_t)(k + u) * n + i0, bl[u], bh[u]);
                }
            }
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                if (k + u < m) {
                    const float ck = c_sh[k + u];
                    const f32x2 ck2 = pk(ck, ck);
#pragma unroll
                    for (int p = 0; p < kPairs; ++p) {
                        const f32x2 t = Item::pair(al[u], ah[u], p), gg = Item::pair(bl[u], bh[u], p);
                        sth[p] = add2(sth[p], t);
                        sg[p] = add2(sg[p], gg);
                        acc[p] = fma2(ck2, sub2(sub2(gg, g0[p]), sub2(t, th0[p])), acc[p]);
                    }
                }
            }
        }
        float res[kCols];
        const f32x2 im2 = pk(inv_m, inv_m), tm2 = pk(-tau * inv_m, -tau * inv_m);
#pragma unroll
        for (int p = 0; p < kPairs; ++p) unpk(fma2(tm2, sg[p], fma2(sth[p], im2, acc[p])), res[2 * p], res[2 * p + 1]);
        if (base) {  // Eq. (4) applied to z: the correction is added to z instead of to the means
            uint2 zl, zh;
            load_item(base + i0, zl, zh);
#pragma unroll
            for (int p = 0; p < kPairs; ++p) unpk(add2(Item::pair(zl, zh, p), acc[p]), res[2 * p], res[2 * p + 1]);
        }
        if (sizeof(T) == 4) {
            stg_stream16(out + i0, make_uint4(__float_as_uint(res[0]), __float_as_uint(res[1]), __float_as_uint(res[2]),
                                              __float_as_uint(res[3])));
        } else {
            uint32_t w0, w1;  // cvt.rn.bf16x2.f32 d, a, b: a -> upper half, b -> lower half
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w0) : "f"(res[1]), "f"(res[0]));
            asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w1) : "f"(res[3]), "f"(res[2]));
            asm volatile("st.global.cs.v2.u32 [%0], {%1,%2};" ::"l"(out + i0), "r"(w0), "r"(w1) : "memory");
        }
    }
}

template <typename T>
static cudaError_t launch_combine_t(const T* theta, const T* g, int64_t n, int m, const qn_coef_block* coef, T* out,
                                    const T* base, cudaStream_t st) {
    const bool aligned = (reinterpret_cast<uintptr_t>(theta) % 16 == 0) && (reinterpret_cast<uintptr_t>(g) % 16 == 0) &&
                         (reinterpret_cast<uintptr_t>(out) % 16 == 0) && (reinterpret_cast<uintptr_t>(base) % 16 == 0) &&
                         ((n * (int64_t)sizeof(T)) % 16 == 0);
    const int threads = aligned ? CombineItem<T>::kThreads : kCombineThreads;
    const int64_t nitems = aligned ? n / CombineItem<T>::kCols : n;
    const int64_t want = (nitems + threads - 1) / threads;
    int per_sm = 1;
    const cudaError_t oe =
        aligned ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, combine_vec_kernel<T>, threads, 0)
                : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, combine_kernel<T, false>, threads, 0);
    if (oe != cudaSuccess || per_sm < 1) per_sm = 1;
    // whole waves only: a grid-strided loop gains nothing from a partial last wave
    const int64_t cap = (int64_t)qn_sm_count() * per_sm * 4;
    const int grid = (int)(want < cap ? (want > 0 ? want : 1) : cap);
    if (aligned)
        combine_vec_kernel<T><<<grid, threads, 0, st>>>(theta, g, n, m, coef, out, base);
    else
        combine_kernel<T, false><<<grid, threads, 0, st>>>(theta, g, n, m, coef, out, base);
    return cudaGetLastError();
}

}  // namespace qn

cudaError_t qn_launch_combine(qn_dtype dtype, const void* theta, const void* g, int64_t n, int m,
                              const qn_coef_block* coef, void* theta_new, cudaStream_t st, int* launches,
                              const void* base) {
    cudaError_t e =
        dtype == QN_F32
            ? qn::launch_combine_t(static_cast<const float*>(theta), static_cast<const float*>(g), n, m, coef,
                                   static_cast<float*>(theta_new), static_cast<const float*>(base), st)
            : qn::launch_combine_t(static_cast<const __nv_bfloat16*>(theta), static_cast<const __nv_bfloat16*>(g), n, m,
                                   coef, static_cast<__nv_bfloat16*>(theta_new), static_cast<const __nv_bfloat16*>(base), st);
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}
