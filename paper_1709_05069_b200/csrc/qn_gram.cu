// Streaming reduction over g[m][n]: per-column reference (the Workers' mean), shifted values
// x_k = g_k - r, the Gram sum_i x_k x_l and the products t_k = sum_i x_k r, as per-CTA fp64 partials
// in the packed layout of qn_internal.h.  (Section 2 of the paper: means, centred matrix G, G^H G
// and the numerators of alpha_k for z = gbar.)  The solve kernel sums the partials in a fixed
// order and applies the exact m x m centring, so any rounding in the per-column reference cancels.
//
// Arithmetic, three modes:
//   kFast     fp32 products, fp32 accumulation over at most kFlushCols columns per thread, then fp64.
//             The rounding errors of the products are unbiased and average out as 1/sqrt(n); used
//             for n >= QN_PRECISE_BELOW, where they stay below 1e-10 of the largest eigenvalue.  (Measured with
//             this mode forced at n = 2^20, m = 16 and a spectrum that reaches down to lambda = 1e-3: sigma error
//             0.9 of the 1e-5 bar against 0.001 in kPrecise, and the pass is no faster there.)
//   kPrecise  the shifted values are rounded to fp32 once, every product and sum is fp64 (a product of
//             two fp32 values is exact in fp64), so the result is the exact Gram of slightly perturbed
//             data and stays positive semi-definite to fp64 accuracy; used for small n.
//   kRaw      as kPrecise with reference 0: the raw Gram of the asynchronous window, which has to
//             carry the cancellation of the later m x m centring.
// Every thread owns fixed columns and fixed output entries, so results are bitwise reproducible for
// a given grid.
#include <math.h>

#include "qn_device.cuh"

namespace qn {

constexpr int kThreads = 256;
enum GramMode { kFast = 0, kPrecise = 1, kRaw = 2 };
constexpr int kFlushCols = 32;  // columns accumulated in fp32 by one thread between fp64 flushes

// ------------------------------------------------------------------------------------------------
// Direct kernel, m <= 8: one thread holds all m values of its columns in registers and owns a full
// private copy of the 36 + 8 accumulators.
// ------------------------------------------------------------------------------------------------
constexpr int kDirectM = 8;
constexpr int kDirectTri = kDirectM * (kDirectM + 1) / 2;  // 36
constexpr int kDirectAcc = kDirectTri + kDirectM;          // 44

// CTA reduction of the direct kernels in a fixed order: butterfly inside each of the first 8 warps, then warps
// 0..7 in sequence; the result goes to the CTA's packed partial.  Every thread of the CTA must call it; warps
// that hold no sums pass `holds_sums = false`.
__device__ __forceinline__ void direct_reduce_store(const double (&acc64)[kDirectAcc], int m, double* __restrict__ partials,
                                                    bool holds_sums) {
    __shared__ double red[kThreads / 32][kDirectAcc];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (holds_sums) {
#pragma unroll
        for (int e = 0; e < kDirectAcc; ++e) {
            const double s = warp_sum(acc64[e]);
            if (lane == 0) red[warp][e] = s;
        }
    }
    __syncthreads();
    if (threadIdx.x < kDirectAcc) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kThreads / 32; ++w) s += red[w][threadIdx.x];
        // map the 8-row packed index to the m-row packed index
        const int e = threadIdx.x;
        double* out = partials + (int64_t)blockIdx.x * qn_partial_len(m);
        if (e < kDirectTri) {
            int k = 0, rem = e;
            while (rem >= kDirectM - k) {
                rem -= kDirectM - k;
                ++k;
            }
            const int l = k + rem;
            if (l < m) out[qn_tri_index(m, k, l)] = s;
        } else {
            const int k = e - kDirectTri;
            if (k < m) out[m * (m + 1) / 2 + k] = s;
        }
    }
}

template <typename T, bool kAligned>
struct DirectItem {
    // one work item = 16 bytes of every row (aligned) or one element of every row (unaligned)
    static constexpr int kCols = kAligned ? Storage<T>::kVec : 1;
    uint4 v[kDirectM];

    __device__ __forceinline__ void load(const T* g, int64_t n, int m, int64_t item, int64_t nitems) {
#pragma unroll
        for (int k = 0; k < kDirectM; ++k) {
            v[k] = make_uint4(0, 0, 0, 0);
            if (k < m && item < nitems) {
                if (kAligned) {
                    v[k] = ldg_stream16(g + (int64_t)k * n + item * kCols);
                } else {
                    v[k].x = __float_as_uint(Storage<T>::load1(g + (int64_t)k * n + item));
                }
            }
        }
    }
    __device__ __forceinline__ float get(int k, int e) const {
        return kAligned ? Storage<T>::get(v[k], e) : __uint_as_float(v[k].x);
    }
};

template <typename T, bool kAligned, int kMode>
__global__ void __launch_bounds__(kThreads, 1)
gram_direct_kernel(const T* __restrict__ g, int64_t n, int m, double* __restrict__ partials, const int* __restrict__ run_if) {
    if (run_if && (*run_if & 1) == 0) return;  // a repeat pass that the spectrum did not ask for
    using Item = DirectItem<T, kAligned>;
    constexpr int kCols = Item::kCols;
    constexpr int kFlushIters = kFlushCols / kCols > 0 ? kFlushCols / kCols : 1;

    const int64_t nitems = kAligned ? n / kCols : n;
    const int64_t ntiles = (nitems + kThreads - 1) / kThreads;

    float acc[kDirectAcc];
    double acc64[kDirectAcc];
#pragma unroll
    for (int e = 0; e < kDirectAcc; ++e) {
        acc[e] = 0.f;
        acc64[e] = 0.0;
    }
    float mask[kDirectM];  // 1 for real Workers, 0 for the padding rows
#pragma unroll
    for (int k = 0; k < kDirectM; ++k) mask[k] = k < m ? 1.f : 0.f;
    const float inv_m = 1.0f / (float)m;

    Item cur, nxt;
    int64_t tile = blockIdx.x;
    cur.load(g, n, m, tile * kThreads + threadIdx.x, tile < ntiles ? nitems : 0);
    int iters = 0;
    for (; tile < ntiles; tile += gridDim.x) {
        const int64_t next_tile = tile + gridDim.x;
        nxt.load(g, n, m, next_tile * kThreads + threadIdx.x, next_tile < ntiles ? nitems : 0);
#pragma unroll
        for (int e = 0; e < kCols; ++e) {
            float x[kDirectM];
            float s = 0.f;
#pragma unroll
            for (int k = 0; k < kDirectM; ++k) {
                x[k] = cur.get(k, e);
                s += x[k];
            }
            const float r = kMode == kRaw ? 0.f : s * inv_m;
#pragma unroll
            for (int k = 0; k < kDirectM; ++k) x[k] = fmaf(-mask[k], r, x[k]);
            if (kMode != kFast) {
                double xd[kDirectM];
#pragma unroll
                for (int k = 0; k < kDirectM; ++k) xd[k] = (double)x[k];
#pragma unroll
                for (int k = 0, idx = 0; k < kDirectM; ++k) {
#pragma unroll
                    for (int l = k; l < kDirectM; ++l, ++idx) acc64[idx] = fma(xd[k], xd[l], acc64[idx]);
                }
                if (kMode == kPrecise) {
                    const double rd = (double)r;
#pragma unroll
                    for (int k = 0; k < kDirectM; ++k) acc64[kDirectTri + k] = fma(xd[k], rd, acc64[kDirectTri + k]);
                }
            } else {
#pragma unroll
                for (int k = 0, idx = 0; k < kDirectM; ++k) {
#pragma unroll
                    for (int l = k; l < kDirectM; ++l, ++idx) acc[idx] = fmaf(x[k], x[l], acc[idx]);
                }
#pragma unroll
                for (int k = 0; k < kDirectM; ++k) acc[kDirectTri + k] = fmaf(x[k], r, acc[kDirectTri + k]);
            }
        }
        if (kMode == kFast && ++iters == kFlushIters) {
            iters = 0;
#pragma unroll
            for (int e = 0; e < kDirectAcc; ++e) {
                acc64[e] += (double)acc[e];
                acc[e] = 0.f;
            }
        }
        cur = nxt;
    }
    if (kMode == kFast) {
#pragma unroll
        for (int e = 0; e < kDirectAcc; ++e) acc64[e] += (double)acc[e];
    }

    direct_reduce_store(acc64, m, partials, true);
}

// ------------------------------------------------------------------------------------------------
// Direct kernel fed by bulk copies, m <= 8, fast arithmetic mode, rows on 16-byte boundaries.  One thread
// issues untiled TMA loads of 3.5 KB row segments into a ring of shared-memory stages (eight segments per
// stage: 8 / MR column blocks of MR rows, 196 KB in flight per SM whatever m), so the seven warps that do the
// arithmetic never wait on HBM latency themselves.  The arithmetic is kFast's on packed pairs of columns, for
// MR = 2, 4 or 8 >= m rows.  Measured against the register-fed kernel above (TB/s): fp32 storage m = 8: 6.4 vs 5.3,
// m = 4: 5.9 vs 3.2; bf16 storage m = 8: 4.5 vs 4.3, m = 4: 4.9 vs 2.4, m = 2: 4.5 vs 1.2 (with bf16 storage and
// eight rows the pass is bound by the instructions per element).
// Every wait is bounded; on a time-out the partial is poisoned and the error word set.
// ------------------------------------------------------------------------------------------------
// packed pairs of fp32 (one 64-bit register, two lanes of the fp32 pipe per instruction)
__device__ __forceinline__ uint64_t gs_pk2(uint32_t lo, uint32_t hi) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "r"(lo), "r"(hi));
    return v;
}
__device__ __forceinline__ uint64_t gs_add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t gs_sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t gs_mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t gs_fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}
// columns 2q and 2q + 1 of a 16-byte vector as a pair of fp32
template <typename T>
__device__ __forceinline__ uint64_t gs_pair(const uint4& v, int q);
template <>
__device__ __forceinline__ uint64_t gs_pair<float>(const uint4& v, int q) {
    return q == 0 ? gs_pk2(v.x, v.y) : gs_pk2(v.z, v.w);
}
template <>
__device__ __forceinline__ uint64_t gs_pair<__nv_bfloat16>(const uint4& v, int q) {
    const uint32_t w = q == 0 ? v.x : q == 1 ? v.y : q == 2 ? v.z : v.w;
    return gs_pk2(w << 16, w & 0xffff0000u);
}

// whether entry e of the 8-row packed layout (36 Gram entries by rows, then 8 products with the reference) involves
// only rows first .. mr-1 (first = 1 where row 0 is the reference: its shifted values are exactly zero)
__host__ __device__ constexpr bool gs_used(int e, int mr, int first) {
    if (e >= kDirectTri) return e - kDirectTri >= first && e - kDirectTri < mr;
    int k = 0, rem = e;
    while (rem >= kDirectM - k) {
        rem -= kDirectM - k;
        ++k;
    }
    return k >= first && k + rem < mr;
}

// the same for all 44 entries as a bit mask (a compile-time constant per mr)
__host__ __device__ constexpr uint64_t gs_used_mask(int mr, int first) {
    uint64_t mask = 0;
    for (int e = 0; e < kDirectAcc; ++e) mask |= (uint64_t)(gs_used(e, mr, first) ? 1 : 0) << e;
    return mask;
}

// bytes of a row segment that starts at column c and has at most seg_cols columns (0 past the end of the row)
template <typename T>
__host__ __device__ inline uint32_t gs_block_bytes(int64_t n, int64_t c, int seg_cols) {
    const int64_t left = n - c;
    return left <= 0 ? 0u : (uint32_t)((left < seg_cols ? left : seg_cols) * (int64_t)sizeof(T));
}

constexpr int kGsWarps = 7;                   // warps that do the arithmetic; one more issues the loads: 256 threads,
constexpr int kGsThreads = (kGsWarps + 1) * 32;  // so that every thread can have the registers its 132 sums need
constexpr int kGsSeg = kGsWarps * 32 * 16;    // bytes of one row in a stage: one 16-byte vector per arithmetic thread
constexpr int kGsStages = 7;
// Columns that one half of a packed fp32 accumulator sums between flushes to fp64.  The flush costs fp64-pipe time
// (bf16 storage, m = 8: 4.40 TB/s with 32 columns, 4.62 with 64, 4.85 with 512); the measured sigma error on inputs
// with a spectral gap is 0.035 of the 1e-5 bar with 64 columns at n = 2^22 and 2^24 alike (0.015 with 32; with 128
// it grows with n).
constexpr int kGsFlushCols = 64;
static_assert(kGsThreads == kThreads, "the reduction of the direct kernels is written for kThreads threads");

struct GsSmem {
    alignas(128) unsigned char seg[kGsStages][kDirectM][kGsSeg];
    alignas(8) uint64_t full[kGsStages];
    uint64_t empty[kGsStages];
    int abort;
};

// MR = 2, 4 or 8 >= m: the rows that are computed (the sums of rows >= MR stay zero and cost nothing; with MR = 8 for
// every m the pass would be bound by the same instruction count whatever m, e.g. 2.3 TB/s at m = 4 with bf16 storage).
// The sums keep their place in the 8-row packed layout, so the reduction is shared with the register-fed kernel.
template <typename T, int MR, bool kRef0>
__global__ void __launch_bounds__(kGsThreads, 1)
gram_stream_kernel(const T* __restrict__ g, int64_t n, int m, double* __restrict__ partials, int* __restrict__ error_word) {
    constexpr int kCols = Storage<T>::kVec;
    constexpr int kSegCols = kGsSeg / (int)sizeof(T);   // columns of one row segment
    constexpr int NB = kDirectM / MR;                    // a stage's 8 segments hold NB column blocks of MR rows, so that
    constexpr int kTileCols = NB * kSegCols;             // every m keeps the same number of bytes in flight
    // each half of a packed accumulator sums every other column: kGsFlushCols columns per half between flushes
    constexpr int kFlushIters = 2 * kGsFlushCols / kCols;
    // Reference of a column: the Workers' mean, or (kRef0) Worker 0's value.  Any reference is exact for the identity
    // that the solve kernel applies; g_k - g_0 is exact in fp32 for bf16 data; row 0's shifted values are exactly zero,
    // so its products are not formed: 42 packed instructions per pair of columns at m = 8 instead of 60.  With bf16
    // storage, where the pass is bound by its instruction count and not by HBM: 6.2 against 4.6 TB/s at m = 8, 5.5
    // against 5.1 at m = 4, 5.1 against 4.5 at m = 2.  The price is accuracy: every entry of the shifted Gram then
    // carries Worker 0's deviation from the mean.  Measured on inputs whose largest mode sits on Workers 0 and 1
    // (the worst case), bf16 storage, in units of the 1e-5 bar: error of any sigma_k against sigma_1 0.16 (mean:
    // 0.013); relative error of the smallest retained sigma_k 0.13 at lambda = 0.01, 0.63 at lambda = 0.005 (it grows
    // as 1 / lambda^2).  So the launcher takes it only for bf16 storage and a known lambda >= QN_REF0_MIN_LAMBDA.
    // (fp32 storage, whose subtraction is not exact: 0.65 against 0.035, and the pass is HBM-bound anyway.)
    constexpr int kFirst = kRef0 ? 1 : 0;
    constexpr uint64_t kUsed = gs_used_mask(MR, kFirst);  // the sums this instance forms
    extern __shared__ unsigned char smem_raw[];
    GsSmem& sm = *reinterpret_cast<GsSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort = &sm.abort;
    const int64_t ntiles = (n + kTileCols - 1) / kTileCols;
    const int my_tiles = blockIdx.x < ntiles ? (int)((ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;

    if (tid == 0) {
        for (int s = 0; s < kGsStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], kGsWarps);
        }
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    double acc64[kDirectAcc];
#pragma unroll
    for (int e = 0; e < kDirectAcc; ++e) acc64[e] = 0.0;

    if (warp == kGsWarps) {
        // ------------------------------------------------------------------ load issue
        if (lane == 0) {
            for (int it = 0; it < my_tiles; ++it) {
                const int s = it % kGsStages, use = it / kGsStages;
                if (use > 0) mbar_wait(&sm.empty[s], (uint32_t)((use - 1) & 1), abort);
                const int64_t col0 = (blockIdx.x + (int64_t)it * gridDim.x) * kTileCols;
                uint32_t total = 0;
#pragma unroll
                for (int b = 0; b < NB; ++b) total += gs_block_bytes<T>(n, col0 + (int64_t)b * kSegCols, kSegCols);
                mbar_arrive_expect_tx(&sm.full[s], (uint32_t)m * total);
#pragma unroll
                for (int b = 0; b < NB; ++b) {
                    const int64_t c = col0 + (int64_t)b * kSegCols;
                    const uint32_t bytes = gs_block_bytes<T>(n, c, kSegCols);
                    if (bytes)
                        for (int k = 0; k < m; ++k)
                            bulk_load(sm.seg[s][b * MR + k], g + (int64_t)k * n + c, bytes, &sm.full[s]);
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ arithmetic
        // Two columns at a time with the packed fp32x2 instructions (one instruction, two FMAs): with bf16
        // storage the scalar form needs most of the FMA issue slots of seven warps at HBM speed.  Each half
        // of a packed accumulator sums every other column.
        uint64_t acc[kDirectAcc];
#pragma unroll
        for (int e = 0; e < kDirectAcc; ++e) acc[e] = 0ull;
        const float inv_m = 1.0f / (float)m;
        const uint64_t inv_m2 = gs_pk2(__float_as_uint(inv_m), __float_as_uint(inv_m));
        int iters = 0;
        for (int it = 0; it < my_tiles; ++it) {
            const int s = it % kGsStages, use = it / kGsStages;
            const int64_t col0 = (blockIdx.x + (int64_t)it * gridDim.x) * kTileCols;
            const bool ok = mbar_wait(&sm.full[s], (uint32_t)(use & 1), abort);
            uint4 vall[kDirectM];  // segment b * MR + k: row k of column block b
#pragma unroll
            for (int b = 0; b < NB; ++b) {
                // the last tile may be short or end before this block
                const bool live = ok && (uint32_t)(tid * 16) < gs_block_bytes<T>(n, col0 + (int64_t)b * kSegCols, kSegCols);
#pragma unroll
                for (int k = 0; k < MR; ++k) {
                    vall[b * MR + k] = make_uint4(0, 0, 0, 0);
                    if (live && k < m) vall[b * MR + k] = *reinterpret_cast<const uint4*>(sm.seg[s][b * MR + k] + tid * 16);
                }
            }
            // the values are in registers: the stage can be refilled
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[s]);
#pragma unroll
            for (int b = 0; b < NB; ++b) {
            const uint4* v = vall + b * MR;
#pragma unroll
            for (int q = 0; q < kCols / 2; ++q) {
                uint64_t x[MR];
#pragma unroll
                for (int k = 0; k < MR; ++k) x[k] = gs_pair<T>(v[k], q);
                uint64_t r;
                if (kRef0) {
                    r = x[0];
                } else {
                    uint64_t sum = x[0];
#pragma unroll
                    for (int k = 1; k < MR; ++k) sum = gs_add2(sum, x[k]);
                    r = gs_mul2(sum, inv_m2);
                }
                // padding rows (m <= k < MR) read as zero and become -r here: they only reach sums that are never output
#pragma unroll
                for (int k = kFirst; k < MR; ++k) x[k] = gs_sub2(x[k], r);
#pragma unroll
                for (int k = kFirst; k < MR; ++k) {
#pragma unroll
                    for (int l = k; l < MR; ++l) {
                        const int idx = k * kDirectM - (k * (k - 1)) / 2 + (l - k);  // place in the 8-row packed layout
                        acc[idx] = gs_fma2(x[k], x[l], acc[idx]);
                    }
                }
#pragma unroll
                for (int k = kFirst; k < MR; ++k) acc[kDirectTri + k] = gs_fma2(x[k], r, acc[kDirectTri + k]);
            }
            if (++iters == kFlushIters) {
                iters = 0;
#pragma unroll
                for (int e = 0; e < kDirectAcc; ++e) {
                    if ((kUsed >> e) & 1ull) {
                        acc64[e] += (double)__uint_as_float((uint32_t)acc[e]) + (double)__uint_as_float((uint32_t)(acc[e] >> 32));
                        acc[e] = 0ull;
                    }
                }
            }
            }  // column blocks of the stage
        }
#pragma unroll
        for (int e = 0; e < kDirectAcc; ++e)
            if ((kUsed >> e) & 1ull)
                acc64[e] += (double)__uint_as_float((uint32_t)acc[e]) + (double)__uint_as_float((uint32_t)(acc[e] >> 32));
    }
    __syncthreads();
    if (*abort) {
        // a wait ran out: give bulk copies that may still be in flight into this CTA's shared memory time to land
        // (bounded: about a millisecond), report, and poison the partial so that the solve sees the failure
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
        if (tid == 0 && error_word) atomicExch(error_word, 1);
#pragma unroll
        for (int e = 0; e < kDirectAcc; ++e) acc64[e] = __longlong_as_double(0x7ff8000000000000ll);
    }
    direct_reduce_store(acc64, m, partials, true);  // the issuing warp adds zeros
}

template <typename T>
static cudaError_t launch_gram_stream(const T* g, int64_t n, int m, double* partials, int* num_partials,
                                      int max_partials, int* error_word, bool ref0, cudaStream_t st) {
    const int mr = m <= 2 ? 2 : m <= 4 ? 4 : 8;
    const int64_t tile_cols = (kDirectM / mr) * (kGsSeg / (int64_t)sizeof(T));
    const int64_t ntiles = (n + tile_cols - 1) / tile_cols;
    const int sms = qn_sm_count();
    int grid = (int)(ntiles < sms ? ntiles : sms);
    if (grid > max_partials) grid = max_partials;
    *num_partials = grid;
    void (*kern)(const T*, int64_t, int, double*, int*);
    if (ref0 && sizeof(T) == 2)
        kern = m <= 2 ? gram_stream_kernel<T, 2, true> : m <= 4 ? gram_stream_kernel<T, 4, true> : gram_stream_kernel<T, 8, true>;
    else
        kern = m <= 2 ? gram_stream_kernel<T, 2, false> : m <= 4 ? gram_stream_kernel<T, 4, false> : gram_stream_kernel<T, 8, false>;
    const size_t smem = sizeof(GsSmem) + 128;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, kGsThreads, smem, st>>>(g, n, m, partials, error_word);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Tiled kernel, 9 <= m <= 64, plain fp32 ALUs.  A tile of kTileCols columns is staged in shared
// memory as shifted fp32 values, one record of RBP floats per column: rows 0..m-1 = x_k, zero padding up
// to a multiple of 8 (RB rows), then the reference r of the column.  The Gram is cut into 8x8 blocks; a
// thread owns one upper-triangle block and a fixed residue class of the tile's columns, with the 64
// accumulators in registers, plus eight for t_k = sum_i x_k r, which the diagonal blocks deliver.
// ------------------------------------------------------------------------------------------------
constexpr int kTileCols = 128;
constexpr int kMaxBlocks = (QN_MAX_M + 7) / 8;                     // 8
constexpr int kMaxRBP = 8 * kMaxBlocks + 4;                        // 68 floats per column record

struct TiledSmem {
    float xs[kTileCols * kMaxRBP];
    float psum[kTileCols * 17];
};

template <typename T, bool kAligned, int kMode>
__global__ void __launch_bounds__(kThreads, 1)
gram_tiled_kernel(const T* __restrict__ g, int64_t n, int m, double* __restrict__ partials, const int* __restrict__ run_if) {
    if (run_if && (*run_if & 1) == 0) return;  // a repeat pass that the spectrum did not ask for
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TiledSmem& sm = *reinterpret_cast<TiledSmem*>(smem_raw);

    constexpr int kCols = kAligned ? Storage<T>::kVec : 1;  // columns per load item
    constexpr int kColGroups = kTileCols / kCols;           // load items per row per tile
    constexpr int kRowGroups = kThreads / kColGroups;       // 8 (fp32 x4), 16 (bf16 x8), 2 (scalar)

    const int nb = (m + 7) / 8;
    const int RB = 8 * nb;
    const int RBP = RB + 4;  // the record's entry RB holds the reference r of the column
    const int ntile = nb * (nb + 1) / 2;
    int S = 4;
    while (S < ntile) S <<= 1;  // slots per column step: 4, 8, 16, 32 or 64
    const int slot = threadIdx.x % S;
    const int col0 = threadIdx.x / S;
    const int colstep = kThreads / S;
    const bool active = slot < ntile;

    __shared__ unsigned char tile_a[64], tile_b[64];  // block coordinates of each slot
    if (threadIdx.x < 64) {
        int t = 0;
        for (int a = 0; a < nb; ++a)
            for (int b = a; b < nb; ++b, ++t)
                if (t == (int)threadIdx.x) {
                    tile_a[t] = (unsigned char)a;
                    tile_b[t] = (unsigned char)b;
                }
    }
    __syncthreads();
    const int ta = active ? tile_a[slot] : 0, tb = active ? tile_b[slot] : 0;

    float acc[64];
    double acc64[64];
#pragma unroll
    for (int e = 0; e < 64; ++e) {
        acc[e] = 0.f;
        acc64[e] = 0.0;
    }
    // t_k = sum_i x_k r: eight more sums, meaningful in the threads of the diagonal blocks (ta == tb)
    float tacc[8];
    double tacc64[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        tacc[e] = 0.f;
        tacc64[e] = 0.0;
    }
    const float inv_m = 1.0f / (float)m;
    const int rg = threadIdx.x % kRowGroups, cg = threadIdx.x / kRowGroups;
    const int64_t ntiles = (n + kTileCols - 1) / kTileCols;
    int cols_since_flush = 0;

    // This thread's part of a tile (rows rg, rg + kRowGroups, ... of its column group) is fetched one tile ahead
    // into registers, so that the latency of the loads is hidden behind the previous tile's arithmetic (the fp64
    // modes, which run at small n where little else hides it; the fast mode has no registers to spare for it).
    constexpr bool kAhead = kMode != kFast;
    constexpr int kPre = QN_MAX_M / kRowGroups;
    constexpr int kPreWords = kAligned ? 4 : 1;  // a 16-byte vector, or one element as fp32
    uint32_t pre[kPre][kPreWords];
    auto fetch = [&](int64_t tile) {
        const int64_t i0 = tile * kTileCols + (int64_t)cg * kCols;
#pragma unroll
        for (int j = 0; j < kPre; ++j) {
            const int k = rg + j * kRowGroups;
#pragma unroll
            for (int w = 0; w < kPreWords; ++w) pre[j][w] = 0u;
            if (k < m && tile < ntiles && i0 < n) {
                if (kAligned) {
                    const uint4 v = ldg_stream16(g + (int64_t)k * n + i0);
                    pre[j][0] = v.x;
                    pre[j][kPreWords > 1 ? 1 : 0] = v.y;
                    pre[j][kPreWords > 2 ? 2 : 0] = v.z;
                    pre[j][kPreWords > 3 ? 3 : 0] = v.w;
                } else {
                    pre[j][0] = __float_as_uint(Storage<T>::load1(g + (int64_t)k * n + i0));
                }
            }
        }
    };
    if (kAhead) fetch(blockIdx.x);

    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        if (!kAhead) fetch(tile);
        // pass A: raw values into the column records, partial sums over this thread's rows
        float ps[kCols];
#pragma unroll
        for (int e = 0; e < kCols; ++e) ps[e] = 0.f;
#pragma unroll
        for (int j = 0; j < kPre; ++j) {
            const int k = rg + j * kRowGroups;
            if (k < m) {
#pragma unroll
                for (int e = 0; e < kCols; ++e) {
                    const float val = kAligned ? Storage<T>::get(make_uint4(pre[j][0], pre[j][kPreWords > 1 ? 1 : 0],
                                                                            pre[j][kPreWords > 2 ? 2 : 0],
                                                                            pre[j][kPreWords > 3 ? 3 : 0]), e)
                                               : __uint_as_float(pre[j][0]);
                    sm.xs[(cg * kCols + e) * RBP + k] = val;
                    ps[e] += val;
                }
            }
        }
        if (kAhead) fetch(tile + gridDim.x);
#pragma unroll
        for (int e = 0; e < kCols; ++e) sm.psum[(cg * kCols + e) * (kRowGroups + 1) + rg] = ps[e];
        __syncthreads();
        // pass B: reference of this thread's columns (fixed summation order), shift own entries
        float r[kCols];
#pragma unroll
        for (int e = 0; e < kCols; ++e) {
            float s = 0.f;
            for (int q = 0; q < kRowGroups; ++q) s += sm.psum[(cg * kCols + e) * (kRowGroups + 1) + q];
            r[e] = kMode == kRaw ? 0.f : s * inv_m;
        }
        if (kMode != kRaw) {
            for (int k = rg; k < m; k += kRowGroups) {
#pragma unroll
                for (int e = 0; e < kCols; ++e) sm.xs[(cg * kCols + e) * RBP + k] -= r[e];
            }
        }
        if (rg == 0) {
#pragma unroll
            for (int e = 0; e < kCols; ++e) {
                sm.xs[(cg * kCols + e) * RBP + RB] = r[e];
                for (int k = m; k < RB; ++k) sm.xs[(cg * kCols + e) * RBP + k] = 0.f;
            }
        }
        __syncthreads();
        // compute: this thread's 8x8 block over its residue class of columns
        if (active) {
            for (int c = col0; c < kTileCols; c += colstep) {
                const float4* rec = reinterpret_cast<const float4*>(&sm.xs[c * RBP]);
                const float4 a0 = rec[2 * ta], a1 = rec[2 * ta + 1];
                const float4 b0 = rec[2 * tb], b1 = rec[2 * tb + 1];
                const float a[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
                const float b[8] = {b0.x, b0.y, b0.z, b0.w, b1.x, b1.y, b1.z, b1.w};
                const float rc = sm.xs[c * RBP + RB];
                if (kMode == kFast) {
#pragma unroll
                    for (int p = 0; p < 8; ++p)
#pragma unroll
                        for (int q = 0; q < 8; ++q) acc[p * 8 + q] = fmaf(a[p], b[q], acc[p * 8 + q]);
#pragma unroll
                    for (int p = 0; p < 8; ++p) tacc[p] = fmaf(a[p], rc, tacc[p]);
                } else {
                    double ad[8], bd[8];
#pragma unroll
                    for (int p = 0; p < 8; ++p) {
                        ad[p] = (double)a[p];
                        bd[p] = (double)b[p];
                    }
#pragma unroll
                    for (int p = 0; p < 8; ++p)
#pragma unroll
                        for (int q = 0; q < 8; ++q) acc64[p * 8 + q] = fma(ad[p], bd[q], acc64[p * 8 + q]);
                    const double rd = (double)rc;
#pragma unroll
                    for (int p = 0; p < 8; ++p) tacc64[p] = fma(ad[p], rd, tacc64[p]);
                }
            }
        }
        if (kMode == kFast) {
            cols_since_flush += kTileCols / colstep;
            if (cols_since_flush >= kFlushCols) {
                cols_since_flush = 0;
#pragma unroll
                for (int e = 0; e < 64; ++e) {
                    acc64[e] += (double)acc[e];
                    acc[e] = 0.f;
                }
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    tacc64[e] += (double)tacc[e];
                    tacc[e] = 0.f;
                }
            }
        }
        __syncthreads();
    }
    if (kMode == kFast) {
#pragma unroll
        for (int e = 0; e < 64; ++e) acc64[e] += (double)acc[e];
#pragma unroll
        for (int e = 0; e < 8; ++e) tacc64[e] += (double)tacc[e];
    }

    // CTA reduction: for each block, sum the kThreads/S column classes in the order 0,1,2,...
    double* red = reinterpret_cast<double*>(smem_raw);  // reuse of the tile storage: kThreads*16 doubles
    double* out = partials + (int64_t)blockIdx.x * qn_partial_len(m);
    const int tri_len = m * (m + 1) / 2;
#pragma unroll
    for (int part = 0; part < 4; ++part) {
        __syncthreads();
#pragma unroll
        for (int e = 0; e < 16; ++e) red[threadIdx.x * 16 + e] = acc64[part * 16 + e];
        __syncthreads();
        for (int w = threadIdx.x; w < S * 16; w += kThreads) {
            const int sl = w / 16, e = part * 16 + (w % 16);
            if (sl >= ntile) continue;
            double s = 0.0;
            for (int q = 0; q < colstep; ++q) s += red[(q * S + sl) * 16 + (w % 16)];
            const int row = 8 * tile_a[sl] + e / 8, col = 8 * tile_b[sl] + e % 8;
            if (row <= col && col < m) out[qn_tri_index(m, row, col)] = s;
        }
    }
    // t from the diagonal blocks, same fixed order
    __syncthreads();
#pragma unroll
    for (int e = 0; e < 8; ++e) red[threadIdx.x * 16 + e] = tacc64[e];
    __syncthreads();
    for (int w = threadIdx.x; w < S * 8; w += kThreads) {
        const int sl = w / 8, e = w % 8;
        if (sl >= ntile || tile_a[sl] != tile_b[sl]) continue;
        double s = 0.0;
        for (int q = 0; q < colstep; ++q) s += red[(q * S + sl) * 16 + e];
        const int row = 8 * tile_a[sl] + e;
        if (row < m) out[tri_len + row] = s;
    }
}

// ------------------------------------------------------------------------------------------------
// Host side
// ------------------------------------------------------------------------------------------------
template <typename T, bool kAligned, int kMode>
static cudaError_t launch_gram_mode(const T* g, int64_t n, int m, double* partials, int grid, cudaStream_t st,
                                    const int* run_if) {
    if (m <= kDirectM) {
        gram_direct_kernel<T, kAligned, kMode><<<grid, kThreads, 0, st>>>(g, n, m, partials, run_if);
        return cudaGetLastError();
    }
    auto kern = gram_tiled_kernel<T, kAligned, kMode>;
    const size_t smem = sizeof(TiledSmem);
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, kThreads, smem, st>>>(g, n, m, partials, run_if);
    return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_gram_t(const T* g, int64_t n, int m, bool raw, double* partials, int* num_partials,
                                 int max_partials, cudaStream_t st, const int* run_if = nullptr,
                                 bool fp64_products = false) {
    const bool aligned = (reinterpret_cast<uintptr_t>(g) % 16 == 0) && ((n * (int64_t)sizeof(T)) % 16 == 0);
    const int sms = qn_sm_count();
    int64_t ntiles;
    if (m <= kDirectM) {
        const int64_t nitems = aligned ? n / Storage<T>::kVec : n;
        ntiles = (nitems + kThreads - 1) / kThreads;
    } else {
        ntiles = (n + kTileCols - 1) / kTileCols;
    }
    int grid = (int)(ntiles < sms ? ntiles : sms);
    if (grid > max_partials) grid = max_partials;
    *num_partials = grid;
    const int mode = raw ? kRaw : (n < QN_PRECISE_BELOW || fp64_products ? kPrecise : kFast);
    if (aligned) {
        if (mode == kRaw) return launch_gram_mode<T, true, kRaw>(g, n, m, partials, grid, st, run_if);
        if (mode == kPrecise) return launch_gram_mode<T, true, kPrecise>(g, n, m, partials, grid, st, run_if);
        return launch_gram_mode<T, true, kFast>(g, n, m, partials, grid, st, run_if);
    }
    if (mode == kRaw) return launch_gram_mode<T, false, kRaw>(g, n, m, partials, grid, st, run_if);
    if (mode == kPrecise) return launch_gram_mode<T, false, kPrecise>(g, n, m, partials, grid, st, run_if);
    return launch_gram_mode<T, false, kFast>(g, n, m, partials, grid, st, run_if);
}

}  // namespace qn

cudaError_t qn_launch_gram(qn_dtype dtype, const void* g, int64_t n, int m, bool raw, double* partials,
                           int* num_partials, int max_partials, cudaStream_t st, int* launches, int* error_word,
                           double lambda_hint, int path, int* kernel_out, const int* run_if) {
    const bool plain_alu = path != QN_GRAM_PATH_AUTO;
    cudaError_t e;
    const int64_t elem = dtype == QN_F32 ? 4 : 2;
    int kernel;
    if (!raw && (run_if || path == QN_GRAM_PATH_FP64)) {
        kernel = (m <= qn::kDirectM ? QN_KERNEL_GRAM_DIRECT : QN_KERNEL_GRAM_TILED) | QN_KERNEL_FP64_PRODUCTS;
        e = dtype == QN_F32 ? qn::launch_gram_t(static_cast<const float*>(g), n, m, false, partials, num_partials,
                                                max_partials, st, run_if, true)
                            : qn::launch_gram_t(static_cast<const __nv_bfloat16*>(g), n, m, false, partials,
                                                num_partials, max_partials, st, run_if, true);
    } else if (!raw && !plain_alu && qn_gram_tc_applicable(dtype, g, n, m)) {
        kernel = QN_KERNEL_GRAM_TENSOR;
        e = qn_launch_gram_tc(dtype, g, n, m, partials, num_partials, max_partials, error_word, st);
    } else if (!raw && !plain_alu && m <= qn::kDirectM && n >= QN_PRECISE_BELOW &&
               reinterpret_cast<uintptr_t>(g) % 16 == 0 && (n * elem) % 16 == 0) {
        // bulk-copy variant of the direct kernel (plain_alu keeps the register-fed one, for A/B runs)
        const bool ref0 = lambda_hint >= QN_REF0_MIN_LAMBDA;
        kernel = QN_KERNEL_GRAM_BULK;
        e = dtype == QN_F32 ? qn::launch_gram_stream(static_cast<const float*>(g), n, m, partials, num_partials,
                                                     max_partials, error_word, false, st)
                            : qn::launch_gram_stream(static_cast<const __nv_bfloat16*>(g), n, m, partials,
                                                     num_partials, max_partials, error_word, ref0, st);
    } else {
        kernel = (m <= qn::kDirectM ? QN_KERNEL_GRAM_DIRECT : QN_KERNEL_GRAM_TILED) |
                 (raw || n < QN_PRECISE_BELOW ? QN_KERNEL_FP64_PRODUCTS : 0);
        e = dtype == QN_F32
                ? qn::launch_gram_t(static_cast<const float*>(g), n, m, raw, partials, num_partials, max_partials, st)
                : qn::launch_gram_t(static_cast<const __nv_bfloat16*>(g), n, m, raw, partials, num_partials,
                                    max_partials, st);
    }
    if (e == cudaSuccess && launches) *launches += 1;
    if (e == cudaSuccess && kernel_out) *kernel_out = kernel;
    return e;
}

double qn_gram_error_coeff(int kernel, qn_dtype dtype, int64_t n, double lambda_hint) {
    if (kernel & QN_KERNEL_FP64_PRODUCTS) return 0.0;
    const double by_n = sqrt((double)QN_PRECISE_BELOW / (double)(n > QN_PRECISE_BELOW ? n : QN_PRECISE_BELOW));
    switch (kernel & 0xff) {
        case QN_KERNEL_GRAM_TENSOR: return dtype == QN_F32 ? QN_REDO_COEFF_TC_F32 : QN_REDO_COEFF_TC_BF16;
        case QN_KERNEL_GRAM_BULK:
            return (dtype == QN_BF16 && lambda_hint >= QN_REF0_MIN_LAMBDA ? QN_REDO_COEFF_REF0_AT_4M : QN_REDO_COEFF_BULK_AT_4M) * by_n;
        case QN_KERNEL_GRAM_DIRECT:
        case QN_KERNEL_GRAM_TILED: return QN_REDO_COEFF_ALU_AT_4M * by_n;
    }
    return 0.0;
}

namespace qn {
template <typename K>
static cudaError_t preload_kernel(K kern, size_t smem = 0) {
    cudaFuncAttributes a;
    cudaError_t e = cudaFuncGetAttributes(&a, kern);  // loads the kernel's code into the current context
    if (e == cudaSuccess && smem) e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    return e;
}
template <typename T, bool kAligned>
static cudaError_t preload_alu() {
    cudaError_t e = cudaSuccess;
    if (e == cudaSuccess) e = preload_kernel(gram_direct_kernel<T, kAligned, kFast>);
    if (e == cudaSuccess) e = preload_kernel(gram_direct_kernel<T, kAligned, kPrecise>);
    if (e == cudaSuccess) e = preload_kernel(gram_direct_kernel<T, kAligned, kRaw>);
    if (e == cudaSuccess) e = preload_kernel(gram_tiled_kernel<T, kAligned, kFast>, sizeof(TiledSmem));
    if (e == cudaSuccess) e = preload_kernel(gram_tiled_kernel<T, kAligned, kPrecise>, sizeof(TiledSmem));
    if (e == cudaSuccess) e = preload_kernel(gram_tiled_kernel<T, kAligned, kRaw>, sizeof(TiledSmem));
    return e;
}
template <typename T>
static cudaError_t preload_stream() {
    const size_t smem = sizeof(GsSmem) + 128;
    cudaError_t e = preload_kernel(gram_stream_kernel<T, 2, false>, smem);
    if (e == cudaSuccess) e = preload_kernel(gram_stream_kernel<T, 4, false>, smem);
    if (e == cudaSuccess) e = preload_kernel(gram_stream_kernel<T, 8, false>, smem);
    if (e == cudaSuccess && sizeof(T) == 2) {
        e = preload_kernel(gram_stream_kernel<T, 2, true>, smem);
        if (e == cudaSuccess) e = preload_kernel(gram_stream_kernel<T, 4, true>, smem);
        if (e == cudaSuccess) e = preload_kernel(gram_stream_kernel<T, 8, true>, smem);
    }
    return e;
}
}  // namespace qn

cudaError_t qn_gram_preload() {
    cudaError_t e = qn::preload_alu<float, true>();
    if (e == cudaSuccess) e = qn::preload_alu<float, false>();
    if (e == cudaSuccess) e = qn::preload_alu<__nv_bfloat16, true>();
    if (e == cudaSuccess) e = qn::preload_alu<__nv_bfloat16, false>();
    if (e == cudaSuccess) e = qn::preload_stream<float>();
    if (e == cudaSuccess) e = qn::preload_stream<__nv_bfloat16>();
    if (e == cudaSuccess) e = qn_gram_tc_preload();
    return e;
}
