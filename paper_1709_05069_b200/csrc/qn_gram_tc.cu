// Tensor-core Gram pass for 9 <= m <= 64 and large n (sm_100a: tcgen05.mma with TMEM accumulators).
//
// What it computes is what qn_gram.cu computes (paper, Section 2: the means, the centred columns and
// G^H G, here in reference-shifted form): per column the fp32 mean r of the m Workers' values,
// x_k = g_k - r, C' = sum_i x x^T and t = sum_i x r, as one fp64 partial per CTA.
//
// Why tensor cores: the Gram needs m(m+1) flops per m loaded elements; at m = 32 that already needs
// most of the fp32 FMA peak to keep up with HBM, and at m = 64 (bf16) three times that peak.
//
// How the precision is kept.  Each shifted value (fp32) is split exactly into hi = bf16(x) and
// lo = bf16(x - hi), 16 significant bits in all.  A tile holds the rows [hi_0..hi_MP-1, lo_0..lo_MP-1]
// of 64 columns, K-major with the 128-byte swizzle, and ONE MMA with that tile as both operands gives
// all four blocks hi hi^T, hi lo^T, lo hi^T, lo lo^T; their sum is the Gram of (hi + lo).  One
// tcgen05.mma costs the issuing thread about 65 cycles whatever its shape, so every instruction is
// M = N = 128: for MP = 64 that is one tile, for MP = 32 two tiles (64 rows each) share a stage and
// the instruction computes both diagonal 64 x 64 blocks at once (the off-diagonal blocks are unused).
// bf16 x bf16
// products are exact, but the tensor core adds them to its fp32 accumulator with truncation: measured on
// B200, a chain of L MMA instructions loses about L * 5e-8 of the accumulated value, nearly but not quite
// uniformly over the matrix.  Chains are therefore kept short: after kFlush tiles (4*kFlush instructions)
// the accumulator is drained into fp32 registers with round-to-nearest adds (unbiased), and every 16
// drains those go to fp64.  Measured effect on sigma for inputs with a singular-value gap: relative
// error of the retained sigma_k about 1e-6 (chains of 4 instructions) to 5e-6 (16 instructions).
// t is accumulated by the CUDA cores that build the tiles (fp32 products, fp64 every tile).
//
// Structure (one persistent CTA per SM, warp-specialised):
//   warps 4-7   drain warps: tcgen05.ld their TMEM quadrant (one D row per thread), fold the hi and lo
//               column halves and add into per-thread fp32 accumulators; fp64 in shared memory every 16
//               drains; the two row halves are added at the end
//   warp  3     one lane issues tcgen05.mma / tcgen05.commit
//   others      producer warps: 128-bit global loads -> registers -> mean by shuffles -> hi/lo split
//               -> swizzled st.shared; one K tile (64 columns) per warp at a time, stages double-buffered
// Stages and accumulator buffers are handed over with mbarriers.  Every wait has an iteration limit:
// when it runs out the CTA sets an abort flag and an error word, stops waiting, finishes its loops,
// frees its TMEM and returns; its partial is poisoned with NaN so the solve reports the failure.
#include "qn_device.cuh"

namespace qn {

// Shape per operand size.  A stage is always 128 rows x 64 columns (16 KB): one tile for MP = 64, two
// tiles for MP = 32.  A producer warp may run ahead of the MMA warp by at most one use of a stage (an
// mbarrier parity wait cannot tell phase k from phase k+2); with in-order consumption that holds as
// long as a warp's next tile lies no more than kStages stages ahead, i.e. kProducers <= kStages*kTilesPerStage.
template <int MP>
struct TcShape {
    static constexpr int kTilesPerStage = MP == 32 ? 2 : 1;
    static constexpr int kProducers = 11;
    static constexpr int kStages = MP == 32 ? 10 : 8;
    static constexpr int kThreads = (4 + 1 + kProducers) * 32;
};

// Stages accumulated in TMEM between drains.  A drain's TMEM loads queue behind the MMAs already issued,
// so very frequent drains stall the MMA thread; very long chains lose accuracy (see the header).  MP = 32:
// every 2 stages (each tile's block then sees chains of 8 instructions); MP = 64: every 4 stages for bf16
// storage, every 2 for fp32 storage, whose inputs carry more bits below the hi/lo split.
template <typename T, int MP>
struct TcFlush {
    static constexpr int kStagesPerDrain = 2;
};
constexpr int kTcTileCols = 64;       // K extent of one tile: 64 bf16 = one 128-byte swizzled row
constexpr int kTcWideEvery = 16;      // drains between fp32 -> fp64 flushes
constexpr uint32_t kTcWaitLimit = 1u << 24;  // polls per wait before giving up (each poll may suspend ~1 us)

template <int MP>
struct TcSmem {
    static constexpr int kStages = TcShape<MP>::kStages;
    static constexpr int kProducers = TcShape<MP>::kProducers;
    alignas(1024) unsigned char stage[kStages][128 * 128];
    double acc64[MP * 128];  // [Gram column][D row], fp64 sums of the folded rows
    alignas(8) uint64_t full[kStages];
    uint64_t done[kStages];  // one per group of stages (only the first kStages / group size are used)
    uint64_t accempty[4];
    uint32_t tmem_base;
    int abort;
};

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
    for (uint32_t it = 0; it < kTcWaitLimit; ++it) {
        if (mbar_try(bar, parity)) return true;
        // waiting producer and drain warps sleep between polls so that they do not take issue slots from
        // the MMA warp; the MMA warp itself polls without sleeping
        if (kBackOff) __nanosleep(64);
        if ((it & 255u) == 255u && *abort) return false;
    }
    *abort = 1;
    return false;
}

// K-major, 128-byte swizzle, 8-row groups 1024 bytes apart (the tile built by the producer warps).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;              // leading byte offset: unused for this layout
    d |= (uint64_t)(1024 >> 4) << 32;    // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;              // descriptor version of sm_100
    d |= (uint64_t)2 << 61;              // 128-byte swizzle
    return d;
}

__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo_elem, float hi_elem) {
    uint32_t w;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(hi_elem), "f"(lo_elem));
    return w;
}

// Packed pairs of fp32 (one 64-bit register, two lanes of the fp32 pipe per instruction).
__device__ __forceinline__ uint64_t pk2(float lo, float hi) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "f"(lo), "f"(hi));
    return v;
}
__device__ __forceinline__ void unpk2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}

// 16 consecutive fp32 columns of this thread's TMEM lane into r[0..15]
#define TC_LD16(r, taddr)                                                                                      \
    asm volatile(                                                                                              \
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                                              \
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"                                      \
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),    \
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]) \
        : "r"(taddr)                                                                                           \
        : "memory")

template <typename T, int MP>
__global__ void __launch_bounds__(TcShape<MP>::kThreads, 1)
gram_tc_kernel(const T* __restrict__ g, int64_t n, int m, double* __restrict__ partials, int* __restrict__ error_word) {
    using Smem = TcSmem<MP>;
    constexpr int RT = 2 * MP;                               // operand rows of one tile: hi rows, then lo rows
    constexpr int U = TcShape<MP>::kTilesPerStage;           // tiles sharing a 128-row stage
    constexpr int kStages = TcShape<MP>::kStages;
    constexpr int kProducers = TcShape<MP>::kProducers;
    constexpr int kDrainEvery = TcFlush<T, MP>::kStagesPerDrain;  // stages per group = per accumulation chain
    constexpr int kGroups = kStages / kDrainEvery;                // groups in the shared-memory ring
    static_assert(kStages % kDrainEvery == 0, "the ring holds whole groups");
    constexpr int LD = sizeof(T) == 2 ? 1 : 2;  // 16-byte registers per 8-column chunk of one row
    constexpr uint32_t kTmemCols = 512;  // four accumulator buffers of 128 fp32 columns: all of TMEM
    constexpr int kAccBufs = 4;
    static_assert(U * RT == 128, "a stage is 128 operand rows");

    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort = &sm.abort;
    // Roles by warp: 3 = MMA issue (alone with one drain and one producer warp on its scheduler), 4..7 = drain
    // (TMEM quadrant = warp - 4 = warp % 4), the rest = producers.
    constexpr int kMmaWarp = 3, kDrainWarp0 = 4;
    const bool is_drain = warp >= kDrainWarp0 && warp < kDrainWarp0 + 4;

    // Tiles of 64 columns are dealt round-robin to the CTAs; a CTA's tiles are grouped U per stage, and
    // the count is padded to a multiple of U with all-zero tiles (they add nothing).
    const int64_t ntiles = (n + kTcTileCols - 1) / kTcTileCols;
    const int64_t my_tiles = blockIdx.x < ntiles ? (ntiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
    constexpr int H = MP / 32;  // producer work items (32 Workers x 64 columns) per tile
    const int64_t my_stages = (my_tiles + U - 1) / U;
    const int64_t my_items_padded = my_stages * 2;  // a stage is two items; a missing one is all zeros
    const int64_t ndrain = (my_stages + kDrainEvery - 1) / kDrainEvery;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.full[s], 2);
            mbar_init(&sm.done[s], 1);
        }
        for (int b = 0; b < kAccBufs; ++b) {
            mbar_init(&sm.accempty[b], 4);
        }
        sm.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sm.tmem_base)),
                     "r"(kTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // operand rows >= m (hi and lo) are never written by the producers and must read as zero
    for (int o = tid * 16; o < kStages * 128 * 128; o += TcShape<MP>::kThreads * 16)
        *reinterpret_cast<uint4*>(&sm.stage[0][0] + o) = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sm.tmem_base;

    if (is_drain) {
        // ------------------------------------------------------------------ drain warps
        const int dq = warp - kDrainWarp0;  // TMEM quadrant of this warp
        const int dtid = dq * 32 + lane;
        // D is 128 x 128 (M = 128: row i in TMEM lane i).  Row r belongs to tile r / RT of the stage and
        // needs that tile's own RT columns only: D[r][cb + c] (hi columns) + D[r][cb + MP + c] (lo columns).
        const int row = dtid;
        const uint32_t cb = (uint32_t)((row / RT) * RT);
        float facc[MP];
#pragma unroll
        for (int e = 0; e < MP; ++e) facc[e] = 0.f;
#pragma unroll 4
        for (int e = 0; e < MP; ++e) sm.acc64[e * 128 + row] = 0.0;
        const int ndrains = (int)ndrain;
        int b = 0, since_wide = 0, gs = 0;
        uint32_t done_par = 0;
        for (int f = 0; f < ndrains; ++f) {
            mbar_wait(&sm.done[gs], done_par, abort);  // the group's MMAs have completed
            __syncwarp();
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            // 32 Gram columns per round: hi and lo halves, four 16-column loads in flight, one wait
#pragma unroll
            for (int c0 = 0; c0 < MP; c0 += 32) {
                uint32_t v0[16], v1[16], u0[16], u1[16];
                const uint32_t taddr = tmem_base + ((uint32_t)(dq * 32) << 16) + (uint32_t)(b * 128) + cb + c0;
                TC_LD16(v0, taddr);
                TC_LD16(v1, taddr + 16);
                TC_LD16(u0, taddr + MP);
                TC_LD16(u1, taddr + MP + 16);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int jj = 0; jj < 16; ++jj) {
                    facc[c0 + jj] += __uint_as_float(v0[jj]) + __uint_as_float(u0[jj]);
                    facc[c0 + 16 + jj] += __uint_as_float(v1[jj]) + __uint_as_float(u1[jj]);
                }
            }
            // the accumulator buffer is free again as soon as every drain warp has read it
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.accempty[b]);
            if (++b == kAccBufs) b = 0;
            if (++gs == kGroups) {
                gs = 0;
                done_par ^= 1u;
            }
            if (++since_wide == kTcWideEvery || f == ndrains - 1) {
                since_wide = 0;
#pragma unroll
                for (int e = 0; e < MP; ++e) {
                    sm.acc64[e * 128 + row] += (double)facc[e];
                    facc[e] = 0.f;
                }
            }
        }
    } else if (warp == kMmaWarp) {
        // ------------------------------------------------------------------ MMA issue
        if (lane == 0) {
            // kind::f16, fp32 accumulate, bf16 x bf16, both K-major, N = 128, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(128 >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            // One thread runs this loop and every instruction in it is on the critical path of the whole
            // CTA, so stage index, parities and descriptors are carried along instead of recomputed.
            const uint64_t desc0 = tc_smem_desc(smem_u32(sm.stage[0]));
            const int nstages = (int)my_stages;
            int s = 0, b = 0, in_chain = 0, gs = 0;
            uint32_t full_par = 0, acc_par = 0;
            for (int p = 0; p < nstages; ++p) {
                const bool first = in_chain == 0;
                if (first) {
                    mbar_wait<false>(&sm.accempty[b], acc_par ^ 1u, abort);
                    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                }
                mbar_wait<false>(&sm.full[s], full_par, abort);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                // the start-address field counts 16-byte units: a stage is 16 KB, a K step of 16 bf16 is 32 B
                const uint64_t desc = desc0 + (uint64_t)(s * (16384 >> 4));
                const uint32_t d_tmem = tmem_base + (uint32_t)(b * 128);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const uint32_t accumulate = (first && k == 0) ? 0u : 1u;
                    asm volatile(
                        "{\n .reg .pred p;\n setp.ne.u32 p, %4, 0;\n"
                        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
                        "l"(desc + 2 * k), "l"(desc + 2 * k), "r"(idesc), "r"(accumulate)
                        : "memory");
                }
                // One commit per group: a commit stalls the tensor pipe for about 430 cycles, so the same
                // mbarrier tells the producers that the group's stages are free and the drain warps that
                // the group's accumulator is complete.
                if (++in_chain == kDrainEvery || p == nstages - 1) {
                    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                                     smem_u32(&sm.done[gs]))
                                 : "memory");
                    in_chain = 0;
                    if (++gs == kGroups) gs = 0;
                    if (++b == kAccBufs) {
                        b = 0;
                        acc_par ^= 1u;
                    }
                }
                if (++s == kStages) {
                    s = 0;
                    full_par ^= 1u;
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ producer warps
        // Work item = 32 rows x 64 columns: a whole tile for MP = 32, a row half of a tile for MP = 64;
        // either way a stage takes two items, from two warps.  The warp's lanes are 8 column chunks (8
        // columns each: one whole 64-column row segment per load instruction) x 4 row groups of 8 rows.
        // Rows are independent of one another (the reference is Worker 0's row, read once per item), so
        // an item's registers are reloaded row by row, each as soon as its row has been converted and
        // stored: a warp keeps loads in flight through the conversion without a second set of registers.
        // Rows >= m are never written; the stages are zeroed once at the start.
        const int pw = warp < kMmaWarp ? warp : warp - 5;
        const int rq = lane >> 3, cl = lane & 7;
        uint4 raw[8][LD], ref[LD], ref_next[LD];
        // 8 columns of Worker `row` in the tile that item k belongs to
        auto load_chunk = [&](uint4 (&dst)[LD], int row, int64_t k) {
            const int64_t q = k / H;
            const int64_t i0 = (blockIdx.x + q * (int64_t)gridDim.x) * kTcTileCols + cl * 8;
#pragma unroll
            for (int l = 0; l < LD; ++l) dst[l] = make_uint4(0, 0, 0, 0);
            if (q < my_tiles && i0 < n) {
                // rows are 32-byte aligned and n is a multiple of 8 on this path (see
                // qn_gram_tc_applicable), so an 8-column chunk is never cut by the end of the row
                if (LD == 1)
                    dst[0] = ldg_stream16(g + (int64_t)row * n + i0);
                else
                    ldg_stream32(g + (int64_t)row * n + i0, dst[0], dst[LD - 1]);
            }
        };
        // first Worker of item k's rows
        auto first_row = [&](int64_t k) { return (int)(k % H) * 32 + rq * 8; };
        load_chunk(ref, 0, pw);
#pragma unroll
        for (int j = 0; j < 8; ++j)
            if (first_row(pw) + j < m) load_chunk(raw[j], first_row(pw) + j, pw);
        for (int64_t k = pw; k < my_items_padded; k += kProducers) {
            const int64_t p = k / 2;                 // stage use this item belongs to
            const int s = (int)(p % kStages);
            // operand rows of the item's Worker rows: hi part at hi0 + (row % 32), lo part MP rows further
            const int hi0 = MP == 32 ? (int)(k & 1) * RT : (int)(k & 1) * 32;
            unsigned char* tile = sm.stage[s] + hi0 * 128;
            const int w0 = first_row(k), w0_next = first_row(k + kProducers);
            load_chunk(ref_next, 0, k + kProducers);
            // the stage must have been consumed by the MMAs of its previous use
            mbar_wait(&sm.done[(p / kDrainEvery) % kGroups], (uint32_t)(((p / kStages) & 1) ^ 1), abort);
#pragma unroll
            for (int j = 0; j < 8; ++j) {
                if (w0 + j < m) {
                    uint32_t hw[4], lw[4];
#pragma unroll
                    for (int pp = 0; pp < 4; ++pp) {
                        const float v0 = Storage<T>::get(raw[j][pp / (4 / LD)], (2 * pp) % (8 / LD));
                        const float v1 = Storage<T>::get(raw[j][pp / (4 / LD)], (2 * pp + 1) % (8 / LD));
                        float r0 = Storage<T>::get(ref[pp / (4 / LD)], (2 * pp) % (8 / LD));
                        float r1 = Storage<T>::get(ref[pp / (4 / LD)], (2 * pp + 1) % (8 / LD));
                        if (j == 0 && w0 == 0) r0 = r1 = 0.f;  // operand row 0 carries the reference itself
                        float x0, x1, l0, l1;
                        unpk2(sub2(pk2(v0, v1), pk2(r0, r1)), x0, x1);
                        hw[pp] = pack_bf16x2_rn(x0, x1);
                        unpk2(sub2(pk2(x0, x1), pk2(__uint_as_float(hw[pp] << 16), __uint_as_float(hw[pp] & 0xffff0000u))),
                              l0, l1);
                        lw[pp] = pack_bf16x2_rn(l0, l1);
                    }
                    // this row's registers are free: fetch the same lane's row of the warp's next item into them
                    if (w0_next + j < m) load_chunk(raw[j], w0_next + j, k + kProducers);
                    const int orow = rq * 8 + j;  // operand row within the item; orow & 7 == j
                    const uint32_t off = (uint32_t)(orow * 128 + ((cl ^ j) << 4));
                    *reinterpret_cast<uint4*>(tile + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                    *reinterpret_cast<uint4*>(tile + MP * 128 + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                } else if (w0_next + j < m) {
                    // no such Worker in this item, but there is one in the warp's next item
                    load_chunk(raw[j], w0_next + j, k + kProducers);
                }
            }
#pragma unroll
            for (int l = 0; l < LD; ++l) ref[l] = ref_next[l];
            // make the generic-proxy stores visible to the tensor core, then hand the tile over
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.full[s]);
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    const double qnan = __longlong_as_double(0x7ff8000000000000ll);
    const bool poisoned = *abort != 0;
    double* out = partials + (int64_t)blockIdx.x * qn_partial_len(m);
    if (tid < 128) {
        // F[a][bc]: hi rows and lo rows of the folded accumulators, over the U tiles of a stage.  Operand
        // row 0 is the reference itself, so F[0][bc] = t[bc] and row 0 of C' (Worker 0 minus itself) is 0.
        constexpr int PER = MP * MP / 128;
        const int a = tid % MP, h = tid / MP;
        const int tri = m * (m + 1) / 2;
#pragma unroll 4
        for (int e = 0; e < PER; ++e) {
            const int bc = h * PER + e;
            if (a <= bc && bc < m) {
                double v = 0.0;
#pragma unroll
                for (int u = 0; u < U; ++u) v += sm.acc64[bc * 128 + u * RT + a] + sm.acc64[bc * 128 + u * RT + MP + a];
                if (poisoned) v = qnan;
                if (a == 0) {
                    out[tri + bc] = bc == 0 ? (poisoned ? qnan : 0.0) : v;
                    out[qn_tri_index(m, 0, bc)] = poisoned ? qnan : 0.0;
                } else {
                    out[qn_tri_index(m, a, bc)] = v;
                }
            }
        }
    }
    if (tid == 0 && *abort && error_word) atomicExch(error_word, 1);
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
    }
}

template <typename T, int MP>
static cudaError_t launch_tc(const T* g, int64_t n, int m, double* partials, int grid, int* error_word,
                             cudaStream_t st) {
    auto kern = gram_tc_kernel<T, MP>;
    const size_t smem = sizeof(TcSmem<MP>) + 1024;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, TcShape<MP>::kThreads, smem, st>>>(g, n, m, partials, error_word);
    return cudaGetLastError();
}

}  // namespace qn

bool qn_gram_tc_applicable(qn_dtype dtype, const void* g, int64_t n, int m) {
    const int64_t elem = dtype == QN_F32 ? 4 : 2;
    // every 8-column chunk of a row is fetched with one load: 16 bytes (bf16) or 32 bytes (fp32), aligned
    const int64_t chunk = 8 * elem;
    return m > 8 && m <= QN_MAX_M && n >= QN_PRECISE_BELOW && (reinterpret_cast<uintptr_t>(g) % chunk == 0) &&
           (n % 8 == 0);
}

cudaError_t qn_launch_gram_tc(qn_dtype dtype, const void* g, int64_t n, int m, double* partials, int* num_partials,
                              int max_partials, int* error_word, cudaStream_t st) {
    const int sms = qn_sm_count();
    const int64_t ntiles = (n + qn::kTcTileCols - 1) / qn::kTcTileCols;
    int grid = (int)(ntiles < sms ? ntiles : sms);
    if (grid > max_partials) grid = max_partials;
    *num_partials = grid;
    if (dtype == QN_F32) {
        const float* p = static_cast<const float*>(g);
        return m <= 32 ? qn::launch_tc<float, 32>(p, n, m, partials, grid, error_word, st)
                       : qn::launch_tc<float, 64>(p, n, m, partials, grid, error_word, st);
    }
    const __nv_bfloat16* p = static_cast<const __nv_bfloat16*>(g);
    return m <= 32 ? qn::launch_tc<__nv_bfloat16, 32>(p, n, m, partials, grid, error_word, st)
                   : qn::launch_tc<__nv_bfloat16, 64>(p, n, m, partials, grid, error_word, st);
}
