// Asynchronous mode: one Worker's Write replaces column `slot` of the window.  This pass lands the new
// gradient column in the window and computes the one row of the window's RAW Gram that changed,
// S[slot][l] = sum_i gnew[i] * g_l[i] for l = 0..m-1 (with g_slot = gnew), reading m*n elements
// instead of the m*(m+1)/2 dot products of a full recomputation.  (The paper, Section 2, allows an
// update after each Write but does not say what the Server keeps; the window and its raw Gram are
// this library's reading.)
//
// The raw Gram has to carry the cancellation of the later m x m centring.  Two arithmetic modes, as in
// the Gram pass: kPrecise (n < QN_PRECISE_BELOW) forms and adds every product in fp64 (a product of two
// fp32 or bf16 values is exact in fp64); the fast mode adds the products of one work item (4 or 8 columns)
// in fp32 starting from zero and then goes to fp64 -- eight times fewer fp32->fp64 conversions, which is
// what bounds the precise mode; its rounding errors are unbiased and average out as 1/sqrt(n).
// The last CTA to finish adds the per-CTA partial rows in a fixed order and patches row and column
// `slot` of the Gram: no CTA ever waits for another.
//
// Two kernels.  row_kernel keeps its rows in registers (any alignment, both arithmetic modes).  For rows on
// 16-byte boundaries and n >= QN_PRECISE_BELOW, row_stream_kernel moves the data with bulk copies instead: one
// thread per CTA issues untiled TMA loads of 4 KB row segments into a ring of shared-memory stages (about
// 200 KB in flight per SM whatever the occupancy; the register kernel is latency-bound at half the HBM
// bandwidth), eight warps take the products out of shared memory, and the new gradient and parameter columns
// are landed in the window by bulk stores straight from the stage, so qn_push needs no separate copy.
#include "qn_device.cuh"

namespace qn {

constexpr int kRowThreads = 256;
constexpr int kRowBlock = 8;  // window columns handled by one CTA row (blockIdx.y)

template <typename T, bool kAligned, bool kPrecise>
__global__ void __launch_bounds__(kRowThreads)
row_kernel(const T* __restrict__ window_g, const T* __restrict__ g_col, T* __restrict__ window_row_out, int64_t n,
           int m, int slot, double* __restrict__ partials, double* __restrict__ raw_gram, double* __restrict__ dots_out,
           unsigned int* ticket) {
    constexpr int kCols = kAligned ? Storage<T>::kVec : 1;
    const int lb = blockIdx.y * kRowBlock;
    const int64_t nitems = kAligned ? n / kCols : n;

    double acc[kRowBlock];
#pragma unroll
    for (int r = 0; r < kRowBlock; ++r) acc[r] = 0.0;

    for (int64_t item = (int64_t)blockIdx.x * kRowThreads + threadIdx.x; item < nitems;
         item += (int64_t)gridDim.x * kRowThreads) {
        const int64_t i0 = item * kCols;
        uint4 xn, xl[kRowBlock];
        if (kAligned)
            xn = ldg_stream16(g_col + i0);
        else
            xn.x = __float_as_uint(Storage<T>::load1(g_col + i0));
#pragma unroll
        for (int r = 0; r < kRowBlock; ++r) {
            const int l = lb + r;
            xl[r] = make_uint4(0, 0, 0, 0);
            if (l < m) {
                if (l == slot)
                    xl[r] = xn;
                else if (kAligned)
                    xl[r] = ldg_stream16(window_g + (int64_t)l * n + i0);
                else
                    xl[r].x = __float_as_uint(Storage<T>::load1(window_g + (int64_t)l * n + i0));
            }
        }
        if (blockIdx.y == 0 && window_row_out) {  // land the column
            if (kAligned)
                stg_stream16(window_row_out + i0, xn);
            else
                window_row_out[i0] = g_col[i0];
        }
        if (kPrecise) {
#pragma unroll
            for (int e = 0; e < kCols; ++e) {
                const double a = (double)(kAligned ? Storage<T>::get(xn, e) : __uint_as_float(xn.x));
#pragma unroll
                for (int r = 0; r < kRowBlock; ++r) {
                    const double b = (double)(kAligned ? Storage<T>::get(xl[r], e) : __uint_as_float(xl[r].x));
                    acc[r] = fma(a, b, acc[r]);
                }
            }
        } else {
            float part[kRowBlock];
#pragma unroll
            for (int r = 0; r < kRowBlock; ++r) part[r] = 0.f;
#pragma unroll
            for (int e = 0; e < kCols; ++e) {
                const float a = kAligned ? Storage<T>::get(xn, e) : __uint_as_float(xn.x);
#pragma unroll
                for (int r = 0; r < kRowBlock; ++r)
                    part[r] = fmaf(a, kAligned ? Storage<T>::get(xl[r], e) : __uint_as_float(xl[r].x), part[r]);
            }
#pragma unroll
            for (int r = 0; r < kRowBlock; ++r) acc[r] += (double)part[r];
        }
    }

    __shared__ double red[kRowThreads / 32][kRowBlock];
    __shared__ bool is_last;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
    for (int r = 0; r < kRowBlock; ++r) {
        const double s = warp_sum(acc[r]);
        if (lane == 0) red[warp][r] = s;
    }
    __syncthreads();
    if (threadIdx.x < kRowBlock && lb + threadIdx.x < m) {
        double s = 0.0;
#pragma unroll
        for (int w = 0; w < kRowThreads / 32; ++w) s += red[w][threadIdx.x];
        partials[(int64_t)blockIdx.x * m + lb + threadIdx.x] = s;
    }
    // last-CTA-done: publish the partial, take a ticket; the CTA that draws the last ticket reduces
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int total = gridDim.x * gridDim.y;
        const unsigned int t = atomicAdd(ticket, 1u);
        is_last = (t == total - 1);
    }
    __syncthreads();
    if (is_last) {
        __threadfence();
        if (threadIdx.x < m) {
            double s0 = 0.0, s1 = 0.0;
            unsigned int p = 0;
            for (; p + 1 < gridDim.x; p += 2) {
                s0 += __ldcg(&partials[(int64_t)p * m + threadIdx.x]);
                s1 += __ldcg(&partials[(int64_t)(p + 1) * m + threadIdx.x]);
            }
            if (p < gridDim.x) s0 += __ldcg(&partials[(int64_t)p * m + threadIdx.x]);
            const double v = s0 + s1;
            if (dots_out) {
                dots_out[threadIdx.x] = v;
            } else {
                raw_gram[slot * m + threadIdx.x] = v;
                raw_gram[threadIdx.x * m + slot] = v;
            }
        }
        if (threadIdx.x == 0) *ticket = 0;  // ready for the next launch on this stream
    }
}


// ------------------------------------------------------------------------------------------------
// Bulk-copy variant (fast arithmetic mode, aligned rows).
// ------------------------------------------------------------------------------------------------
constexpr int kRsSeg = 4096;      // bytes of one row in a stage: 256 threads x 16 bytes
constexpr int kRsStages = 5;
constexpr int kRsConsumers = 256;
constexpr int kRsThreads = kRsConsumers + 32;  // + one warp whose lane 0 issues the loads
constexpr int kRsSlots = kRowBlock + 2;        // window rows, the new gradient column, the new parameter column

struct RsSmem {
    alignas(128) unsigned char seg[kRsStages][kRsSlots][kRsSeg];
    alignas(8) uint64_t full[kRsStages];
    uint64_t empty[kRsStages];
    double red[kRsConsumers / 32][kRowBlock];
    int abort;
    int is_last;
};

template <typename T>
__global__ void __launch_bounds__(kRsThreads, 1)
row_stream_kernel(const T* __restrict__ window_g, const T* __restrict__ g_col, T* __restrict__ window_row_out,
                  const T* __restrict__ theta_col, T* __restrict__ theta_row_out, int64_t n, int m, int slot,
                  double* __restrict__ partials, double* __restrict__ raw_gram, double* __restrict__ dots_out,
                  unsigned int* ticket, int* __restrict__ error_word) {
    constexpr int kCols = Storage<T>::kVec;                   // columns per 16-byte vector
    constexpr int kTileCols = kRsSeg / (int)sizeof(T);        // columns per stage
    extern __shared__ unsigned char smem_raw[];
    RsSmem& sm = *reinterpret_cast<RsSmem*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~(uintptr_t)127);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort = &sm.abort;
    const int lb = blockIdx.y * kRowBlock;
    const bool lands = blockIdx.y == 0 && window_row_out != nullptr;  // this slice of rows also lands the new columns
    const int64_t ntiles = (n + kTileCols - 1) / kTileCols;
    const int my_tiles = blockIdx.x < ntiles ? (int)((ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x) : 0;

    if (tid == 0) {
        for (int s = 0; s < kRsStages; ++s) {
            mbar_init(&sm.full[s], 1);
            mbar_init(&sm.empty[s], kRsConsumers / 32);
        }
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    double acc[kRowBlock];
#pragma unroll
    for (int r = 0; r < kRowBlock; ++r) acc[r] = 0.0;

    if (warp == kRsConsumers / 32) {
        // ------------------------------------------------------------------ load issue
        if (lane == 0) {
            for (int it = 0; it < my_tiles; ++it) {
                const int s = it % kRsStages, use = it / kRsStages;
                if (use > 0) mbar_wait(&sm.empty[s], (uint32_t)((use - 1) & 1), abort);
                const int64_t col0 = (blockIdx.x + (int64_t)it * gridDim.x) * kTileCols;
                const int64_t left = n - col0;
                const uint32_t bytes = (uint32_t)((left < kTileCols ? left : kTileCols) * (int64_t)sizeof(T));
                int nseg = 1 + (lands && theta_col ? 1 : 0);
#pragma unroll
                for (int r = 0; r < kRowBlock; ++r) nseg += (lb + r < m && lb + r != slot) ? 1 : 0;
                mbar_arrive_expect_tx(&sm.full[s], (uint32_t)nseg * bytes);
#pragma unroll
                for (int r = 0; r < kRowBlock; ++r)
                    if (lb + r < m && lb + r != slot)
                        bulk_load(sm.seg[s][r], window_g + (int64_t)(lb + r) * n + col0, bytes, &sm.full[s]);
                bulk_load(sm.seg[s][kRowBlock], g_col + col0, bytes, &sm.full[s]);
                if (lands && theta_col) bulk_load(sm.seg[s][kRowBlock + 1], theta_col + col0, bytes, &sm.full[s]);
            }
        }
    } else {
        // ------------------------------------------------------------------ products
        for (int it = 0; it < my_tiles; ++it) {
            const int s = it % kRsStages, use = it / kRsStages;
            const int64_t col0 = (blockIdx.x + (int64_t)it * gridDim.x) * kTileCols;
            const int64_t left = n - col0;
            const uint32_t bytes = (uint32_t)((left < kTileCols ? left : kTileCols) * (int64_t)sizeof(T));
            const bool ok = mbar_wait(&sm.full[s], (uint32_t)(use & 1), abort);
            if (lands && tid == 0 && ok) {
                // land the new columns: the stage holds exactly the bytes that go to the window
                bulk_store(window_row_out + col0, sm.seg[s][kRowBlock], bytes);
                if (theta_col) bulk_store(theta_row_out + col0, sm.seg[s][kRowBlock + 1], bytes);
                bulk_store_commit();
            }
            const bool live = ok && (uint32_t)(tid * 16) < bytes;  // the last tile may be short; a failed wait adds nothing
            uint4 xn = make_uint4(0, 0, 0, 0), xl[kRowBlock];
            if (live) xn = *reinterpret_cast<const uint4*>(sm.seg[s][kRowBlock] + tid * 16);
#pragma unroll
            for (int r = 0; r < kRowBlock; ++r) {
                const int l = lb + r;
                xl[r] = make_uint4(0, 0, 0, 0);
                if (l == slot)
                    xl[r] = xn;
                else if (live && l < m)
                    xl[r] = *reinterpret_cast<const uint4*>(sm.seg[s][r] + tid * 16);
            }
            float part[kRowBlock];
#pragma unroll
            for (int r = 0; r < kRowBlock; ++r) part[r] = 0.f;
#pragma unroll
            for (int e = 0; e < kCols; ++e) {
                const float a = Storage<T>::get(xn, e);
#pragma unroll
                for (int r = 0; r < kRowBlock; ++r) part[r] = fmaf(a, Storage<T>::get(xl[r], e), part[r]);
            }
#pragma unroll
            for (int r = 0; r < kRowBlock; ++r) acc[r] += (double)part[r];
            // the stage may be refilled once every warp has read it and the bulk stores have read it
            if (lands && tid == 0) bulk_store_wait_read();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.empty[s]);
        }
        if (lands && tid == 0) bulk_store_wait_all();  // the landed columns are in global memory before the CTA signals
    }

    if (*abort) {
        // a wait ran out: give the bulk copies that may still be in flight into this CTA's shared memory time to
        // land (bounded: about a millisecond) before the CTA returns
#pragma unroll 1
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);
    }
    // CTA reduction in a fixed order, then last-CTA-done as in row_kernel
    if (warp < kRsConsumers / 32) {
#pragma unroll
        for (int r = 0; r < kRowBlock; ++r) {
            const double v = warp_sum(acc[r]);
            if (lane == 0) sm.red[warp][r] = v;
        }
    }
    __syncthreads();
    if (tid < kRowBlock && lb + tid < m) {
        double v = 0.0;
#pragma unroll
        for (int w = 0; w < kRsConsumers / 32; ++w) v += sm.red[w][tid];
        if (*abort) v = __longlong_as_double(0x7ff8000000000000ll);
        partials[(int64_t)blockIdx.x * m + lb + tid] = v;
    }
    if (tid == 0 && *abort && error_word) atomicExch(error_word, 1);
    __threadfence();
    __syncthreads();
    if (tid == 0) {
        const unsigned int total = gridDim.x * gridDim.y;
        const unsigned int t = atomicAdd(ticket, 1u);
        sm.is_last = (t == total - 1);
    }
    __syncthreads();
    if (sm.is_last) {
        __threadfence();
        if (tid < m) {
            double s0 = 0.0, s1 = 0.0;
            unsigned int p = 0;
            for (; p + 1 < gridDim.x; p += 2) {
                s0 += __ldcg(&partials[(int64_t)p * m + tid]);
                s1 += __ldcg(&partials[(int64_t)(p + 1) * m + tid]);
            }
            if (p < gridDim.x) s0 += __ldcg(&partials[(int64_t)p * m + tid]);
            const double v = s0 + s1;
            if (dots_out) {
                dots_out[tid] = v;
            } else {
                raw_gram[slot * m + tid] = v;
                raw_gram[tid * m + slot] = v;
            }
        }
        if (tid == 0) *ticket = 0;  // ready for the next launch on this stream
    }
}

template <typename T>
static cudaError_t launch_row_t(const T* window_g, const T* g_col, T* window_row_out, const T* theta_col,
                                T* theta_row_out, int64_t n, int m, int slot, double* partials, int max_partials,
                                double* raw_gram, double* dots_out, unsigned int* ticket, int* error_word,
                                bool* theta_landed, cudaStream_t st) {
    const bool aligned = (reinterpret_cast<uintptr_t>(window_g) % 16 == 0) &&
                         (reinterpret_cast<uintptr_t>(g_col) % 16 == 0) && ((n * (int64_t)sizeof(T)) % 16 == 0);
    *theta_landed = false;
    if (aligned && n >= QN_PRECISE_BELOW && reinterpret_cast<uintptr_t>(window_row_out) % 16 == 0 &&
        reinterpret_cast<uintptr_t>(theta_col) % 16 == 0 && reinterpret_cast<uintptr_t>(theta_row_out) % 16 == 0) {
        const int nby = (m + kRowBlock - 1) / kRowBlock;
        const int64_t ntiles = (n + kRsSeg / (int64_t)sizeof(T) - 1) / (kRsSeg / (int64_t)sizeof(T));
        int64_t cap = qn_sm_count() / nby;  // one CTA per SM (the stages take most of its shared memory)
        if (cap < 1) cap = 1;
        if (cap > max_partials) cap = max_partials;
        const int gx = (int)(ntiles < cap ? ntiles : cap);
        auto kern = row_stream_kernel<T>;
        const size_t smem = sizeof(RsSmem) + 128;
        cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        kern<<<dim3(gx, nby), kRsThreads, smem, st>>>(window_g, g_col, window_row_out, theta_col, theta_row_out, n, m,
                                                     slot, partials, raw_gram, dots_out, ticket, error_word);
        *theta_landed = theta_col != nullptr;
        return cudaGetLastError();
    }
    const int64_t nitems = aligned ? n / Storage<T>::kVec : n;
    const int nby = (m + kRowBlock - 1) / kRowBlock;
    // one wave of CTAs: every resident slot of every SM gets one CTA (the loop is grid-strided, so a second,
    // partial wave would run at a fraction of the occupancy for as long as the first)
    int per_sm = 1;
    {
        const bool precise_q = n < QN_PRECISE_BELOW;
        cudaError_t oe = aligned && !precise_q
                             ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, row_kernel<T, true, false>, kRowThreads, 0)
                             : aligned ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, row_kernel<T, true, true>, kRowThreads, 0)
                                       : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, row_kernel<T, false, true>, kRowThreads, 0);
        if (oe != cudaSuccess || per_sm < 1) per_sm = 1;
    }
    int64_t want = (nitems + kRowThreads - 1) / kRowThreads;
    int64_t cap = (int64_t)qn_sm_count() * per_sm / nby;
    if (cap < 1) cap = 1;
    if (cap > max_partials) cap = max_partials;
    const int gx = (int)(want < cap ? (want > 0 ? want : 1) : cap);
    dim3 grid(gx, nby);
    const bool precise = n < QN_PRECISE_BELOW;
    if (aligned && !precise)
        row_kernel<T, true, false><<<grid, kRowThreads, 0, st>>>(window_g, g_col, window_row_out, n, m, slot, partials,
                                                                raw_gram, dots_out, ticket);
    else if (aligned)
        row_kernel<T, true, true><<<grid, kRowThreads, 0, st>>>(window_g, g_col, window_row_out, n, m, slot, partials,
                                                               raw_gram, dots_out, ticket);
    else
        row_kernel<T, false, true><<<grid, kRowThreads, 0, st>>>(window_g, g_col, window_row_out, n, m, slot, partials,
                                                                raw_gram, dots_out, ticket);
    return cudaGetLastError();
}

}  // namespace qn

// Self-test of the bounded waits: one warp waits, with the library's own wait routine, on an mbarrier that nothing
// ever arrives on.  The wait runs out after its limit (one second), the CTA reports through the error
// word exactly as the streaming kernels do, and returns; the context stays usable.
namespace qn {
__global__ void __launch_bounds__(32) wait_probe_kernel(int* error_word) {
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    const bool ok = mbar_wait(&bar, 0u, &abort_flag);
    __syncwarp();
    if (threadIdx.x == 0 && !ok && error_word) atomicExch(error_word, 1);
}
}  // namespace qn

cudaError_t qn_launch_wait_probe(int* error_word, cudaStream_t st) {
    qn::wait_probe_kernel<<<1, 32, 0, st>>>(error_word);
    return cudaGetLastError();
}

cudaError_t qn_launch_row(qn_dtype dtype, const void* window_g, const void* g_col, void* window_row_out,
                          const void* theta_col, void* theta_row_out, int64_t n, int m, int slot, double* partials,
                          int max_partials, double* raw_gram, double* dots_out, unsigned int* ticket, int* error_word,
                          bool* theta_landed, cudaStream_t st, int* launches) {
    cudaError_t e =
        dtype == QN_F32
            ? qn::launch_row_t(static_cast<const float*>(window_g), static_cast<const float*>(g_col),
                               static_cast<float*>(window_row_out), static_cast<const float*>(theta_col),
                               static_cast<float*>(theta_row_out), n, m, slot, partials, max_partials, raw_gram,
                               dots_out, ticket, error_word, theta_landed, st)
            : qn::launch_row_t(static_cast<const __nv_bfloat16*>(window_g), static_cast<const __nv_bfloat16*>(g_col),
                               static_cast<__nv_bfloat16*>(window_row_out), static_cast<const __nv_bfloat16*>(theta_col),
                               static_cast<__nv_bfloat16*>(theta_row_out), n, m, slot, partials, max_partials, raw_gram,
                               dots_out, ticket, error_word, theta_landed, st);
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}
