// Tensor-core Gram pass for 9 <= m <= 64 and large n (sm_100a: tcgen05.mma with TMEM accumulators).
//
// What it computes is what qn_gram.cu computes (paper, Section 2: the means, the centred columns and
// G^H G, here in reference-shifted form): per column a reference r close to the mean of the m Workers'
// values, x_k = g_k - r, C' = sum_i x x^T and t = sum_i x r, as one fp64 partial per CTA.  The solve
// kernel's m x m centring is exact for ANY r (G^H G = P C' P, G^H gbar = P t + P C' 1/m), so r only has
// to be near the mean, and it is chosen so that the tensor core sees it without error:
//   bf16 storage: r = the mean formed with packed bf16 adds (a bf16 number); x = g - r is split by an
//                 error-free TwoSum in packed bf16 arithmetic into hi = bf16(g - r) and lo = (g - r) - hi,
//                 so hi + lo is the shifted value EXACTLY and costs six packed instructions per pair.
//   fp32 storage: r = the fp32 mean rounded to 16 significant bits (rh + rl, two bf16 numbers);
//                 x = fl(g - r), hi = bf16(x), lo = bf16(x - hi): 16 significant bits of x.
//
// Why tensor cores: the Gram needs m(m+1) flops per m loaded elements; at m = 32 that already needs
// most of the fp32 FMA peak to keep up with HBM, and at m = 64 (bf16) three times that peak.
//
// Operand layout.  A stage is 144 rows x 64 K-slots of bf16, K-major with the 128-byte swizzle.  Rows
// 0..127 hold U = 64/MP tiles (MP = 16, 32 or 64 >= m): tile u = rows [hi_0..hi_MP-1, lo_0..lo_MP-1] of
// 64 consecutive columns.  Rows 128 + 2u and 129 + 2u hold rh and rl of tile u's columns.  ONE MMA
// (M = 128, N = 144, K = 16) uses rows 0..127 as A and all 144 rows as B: its diagonal 2MP x 2MP blocks
// are the four products hi hi^T, hi lo^T, lo hi^T, lo lo^T of each tile, whose sum is the Gram of
// (hi + lo), and columns 128 + 2u, 129 + 2u give t.  (One tcgen05.mma costs about the same whatever its
// shape up to N = 128, so the blocks off the diagonal are computed and ignored.)
//
// bf16 x bf16 products are exact, but the tensor core adds them to its fp32 accumulator with truncation:
// measured on B200, a chain of L MMA instructions loses about L * 5e-8 of the accumulated value, nearly
// but not quite uniformly over the matrix.  Chains are therefore short: after 2 (fp32 storage) or 4 (bf16
// storage) stages of four instructions each the accumulator is drained into fp32 registers with round-to-nearest adds
// (unbiased), and every kTcWideEvery drains those go to fp64.  The error that is left is proportional to
// the magnitude of the entries of C', which is why the reference is the mean and not one Worker's row.
//
// Structure (one persistent CTA per SM, warp-specialised):
//   warps 4-7   drain warps: tcgen05.ld their TMEM quadrant (one D row per thread), fold the hi and lo
//               column halves and add into per-thread fp32 accumulators (packed pairs); fp64 in shared
//               memory every kTcWideEvery drains
//   warps 3, 9  one lane of each issues tcgen05.mma / tcgen05.commit for every other group of stages
//   others      producer warps: global loads -> registers -> reference -> hi/lo split -> swizzled
//               st.shared.  A work item is 8 KB of g: all MP rows x (512/MP) columns (bf16, a whole stage)
//               or MP rows x (256/MP) columns (fp32, half a stage), so a warp holds every Worker's value
//               of its columns.  An item's registers are reloaded row by row for the warp's next item as
//               soon as a row has been converted, and the item after that is prefetched into L2.
// Stages and accumulator buffers are handed over with mbarriers: full[stage] (producers -> MMA), done[..][group]
// (a commit after every kTcRelease stages -> producers: the group's stages are free), accfull[buffer] (a commit
// at the end of a chain -> drain warps) and accempty[buffer] (drain warps -> MMA).  A parity wait cannot tell
// phase k from phase k + 2.  The two MMA warps complete groups out of order (by up to kTcAccBufs chains), and a
// producer warp's next item may lie more than one revolution of the stage ring ahead of its last one, so a
// producer could meet a "group consumed" barrier two phases behind what it expects; therefore each group has
// FOUR such barriers, used by revolutions 0, 1, 2, 3 (mod 4) of the ring, and a waiter is then never more
// than one phase of ITS barrier off.  The MMA warps cannot get a revolution ahead of the fills they wait for,
// because the previous use of a stage was consumed by the same warp or by a chain that is already drained
// (accempty).  (All of this was checked with a random-schedule simulation of the protocol.)
// Every wait has an iteration limit:
// when it runs out the CTA sets an abort flag and an error word, stops waiting, finishes its loops,
// frees its TMEM and returns; its partial is poisoned with NaN so the solve reports the failure.
#include <type_traits>

#include "qn_device.cuh"

namespace qn {

constexpr int kTcMmaWarps = 2;
#ifndef QN_TC_PRODUCERS_BF16
#define QN_TC_PRODUCERS_BF16 10
#endif
#ifndef QN_TC_PRODUCERS_64
#define QN_TC_PRODUCERS_64 8
#endif
// Warp roles.  Warps 4-7 drain (a warp reads the TMEM lanes of quadrant warp % 4), two warps issue the MMAs, the rest
// convert.  A warp's scheduler is warp % 4.  16 warps, ten producers (3, 2, 3, 2 per scheduler), except bf16 storage
// at MP = 64: the ring holds eight stages, i.e. the items of four teams of two warps, so a fifth team mostly waits for a
// stage, and the conversion is bound by the schedulers' issue rate: 14 warps, eight producers, two on every scheduler
// (measured 3.65 against 3.56 TB/s; registers are allocated to warps in fours, so 14 warps get no more than 16 would).
// fp32 storage at MP = 64 waits for its loads instead and needs the ten warps' bytes in flight (4.4 against 3.7 TB/s).
template <typename T, int MP>
struct TcRoles {
    static constexpr int kProducers = sizeof(T) == 2 ? (MP == 64 ? QN_TC_PRODUCERS_64 : QN_TC_PRODUCERS_BF16) : 10;
    static constexpr bool kEight = kProducers == 8;
    static constexpr int kThreads = (4 + kTcMmaWarps + kProducers) * 32;
    static constexpr int kMmaWarp = kEight ? 12 : 3, kMmaWarpB = kEight ? 13 : 9, kDrainWarp0 = 4;
    // producer index 0 .. kProducers-1 of a warp that neither drains nor issues
    static __device__ __forceinline__ int producer_index(int warp) {
        if (kEight) return warp < 4 ? warp : warp - 4;                    // warps 0-3, 8-11
        return warp < 3 ? warp : warp == 8 ? 3 : warp - 6;                // warps 0-2, 8, 10-15
    }
};
constexpr int kTcStageRows = 144;                 // 128 operand rows + 16 rows for the references (B operand only)
constexpr int kTcStageBytes = kTcStageRows * 128;
constexpr int kTcRelease = 2;                     // stages released to the producers by one commit
constexpr int kTcAccBufs = 3;                     // accumulator buffers in TMEM
constexpr int kTcAccStride = 160;                 // TMEM columns from one buffer to the next (144 used)
constexpr int kTcWideEvery = 16;                  // drains between fp32 -> fp64 flushes
#ifndef QN_TC_RUN_BYTES
#define QN_TC_RUN_BYTES 512
#endif
constexpr int kTcRunBytes = QN_TC_RUN_BYTES;           // bytes of one row that a CTA's consecutive stages cover
#ifndef QN_TC_PREFETCH_BF16
#define QN_TC_PREFETCH_BF16 1
#endif
#ifndef QN_TC_PREFETCH_F32
#define QN_TC_PREFETCH_F32 0
#endif
#ifndef QN_TC_FASTPATH_F32
#define QN_TC_FASTPATH_F32 1
#endif
#ifndef QN_TC_CHAIN_F32
#define QN_TC_CHAIN_F32 2
#endif
#ifndef QN_TC_CHAIN_BF16
#define QN_TC_CHAIN_BF16 4
#endif

template <typename T, int MP>
struct TcShape {
    // Lane layout of a producer warp.  A lane holds 8 consecutive columns (one 16-byte chunk of bf16, one 32-byte
    // chunk of fp32) of kRowsPerLane rows; the lanes that share a row read consecutive chunks, so one load
    // instruction reads >= 256 contiguous bytes of every row it touches (128-byte requests reach a third of
    // the HBM bandwidth, 256-byte ones nearly all of it).  A warp covers min(MP, 32) rows; for MP = 64 two
    // warps (a team) cover the rows of the same columns and exchange their column sums through shared memory.
    static constexpr int kRowsPerLane = sizeof(T) == 2 ? 16 : 8;
    static constexpr int kRowsPerWarp = MP < 32 ? MP : 32;
    static constexpr int kRowGroups = kRowsPerWarp / kRowsPerLane;      // lanes of a warp that share a column chunk
    static constexpr int kChunksPerItem = 32 / kRowGroups;              // 8-column chunks of one work item
    static constexpr int kTeam = MP / kRowsPerWarp;                     // warps that share the columns of an item
    static constexpr int kTeams = TcRoles<T, MP>::kProducers / kTeam;
    static constexpr int kItemCols = 8 * kChunksPerItem;
    static constexpr int kTilesPerStage = 64 / MP;
    static constexpr int kStageCols = 64 * kTilesPerStage;
    static constexpr int kStagesPerItem = kItemCols > kStageCols ? kItemCols / kStageCols : 1;  // 2 for bf16, MP = 64
    static constexpr int kItemsPerStage = kStageCols > kItemCols ? kStageCols / kItemCols : 1;  // 2 for fp32, MP <= 32
    static constexpr int kArrivals = kTeam * kItemsPerStage;            // warps that fill one stage
    // A CTA takes runs of kRun adjacent stages, so that the stages of one item are adjacent in memory.
    static constexpr int kStageRowBytes = kStageCols * (int)sizeof(T);
    static constexpr int kRun = kStageRowBytes >= kTcRunBytes ? 1 : kTcRunBytes / kStageRowBytes;
    static constexpr int kStages = MP == 64 ? 8 : 10;
    static_assert(kRowGroups >= 1 && TcRoles<T, MP>::kProducers % kTeam == 0 && kRun % kStagesPerItem == 0, "shape");
    static_assert(kStagesPerItem <= kTcRelease, "the stages of an item belong to one release group");
    // Stages per accumulation chain = per drain.  The error of a chain grows with its length; bf16 storage
    // (hi + lo exact, no input rounding at all) has the margin for 16 instructions, fp32 storage keeps 8.
    static constexpr int kChainStages = sizeof(T) == 2 ? QN_TC_CHAIN_BF16 : QN_TC_CHAIN_F32;
    static_assert(kStages % kTcRelease == 0 && kChainStages % kTcRelease == 0, "whole release groups");
    static_assert(kTeams * kStagesPerItem <= 2 * kStages * kItemsPerStage, "a warp's consecutive items are at most two revolutions apart");
};

template <int MP>
struct TcSmem {
    static constexpr int kStages = MP == 64 ? 8 : 10;
    alignas(1024) unsigned char stage[kStages][kTcStageBytes];
    double acc64[MP * 128];  // [Gram column][D row], fp64 sums of the folded rows
    double t64[128];         // [D row], fp64 sums of the reference columns
    alignas(8) uint64_t full[kStages];
    uint64_t done[4][kStages];  // [revolution of the ring & 3][group of stages] (the first kStages / kTcRelease are used)
    uint64_t accfull[kTcAccBufs];
    uint64_t accempty[kTcAccBufs];
    uint32_t tmem_base;
    int abort;
    // column sums exchanged by the two warps of a team (MP = 64): [team][item parity][warp of the team][chunk]
    alignas(16) uint4 xbuf[MP == 64 ? 5 : 1][2][2][16][2];
};

// K-major, 128-byte swizzle, 8-row groups 1024 bytes apart (the stage built by the producer warps).
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;              // leading byte offset: unused for this layout
    d |= (uint64_t)(1024 >> 4) << 32;    // stride byte offset between 8-row groups
    d |= (uint64_t)1 << 46;              // descriptor version of sm_100
    d |= (uint64_t)2 << 61;              // 128-byte swizzle
    return d;
}

// ---- packed arithmetic ----------------------------------------------------------------------------
// bf16x2: two bf16 numbers in one 32-bit register, round to nearest even, subnormals kept.
__device__ __forceinline__ uint32_t add_bf2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("add.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t sub_bf2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
__device__ __forceinline__ uint32_t mul_bf2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}
// cvt.rn.bf16x2.f32 d, a, b: a -> upper half, b -> lower half (the lower half is the lower column)
__device__ __forceinline__ uint32_t pack_bf16x2_rn(float lo_elem, float hi_elem) {
    uint32_t w;
    asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(w) : "f"(hi_elem), "f"(lo_elem));
    return w;
}
// f32x2: pairs of fp32 in one 64-bit register, two lanes of the fp32 pipe per instruction.
__device__ __forceinline__ uint64_t pk2(uint32_t lo, uint32_t hi) {
    uint64_t v;
    asm("mov.b64 %0, {%1, %2};" : "=l"(v) : "r"(lo), "r"(hi));
    return v;
}
__device__ __forceinline__ void unpk2(uint64_t v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ uint64_t add2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t sub2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
__device__ __forceinline__ uint64_t mul2(uint64_t a, uint64_t b) {
    uint64_t d;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(d) : "l"(a), "l"(b));
    return d;
}
// the two bf16 halves of w as a pair of fp32
__device__ __forceinline__ uint64_t widen_bf2(uint32_t w) { return pk2(w << 16, w & 0xffff0000u); }
// pair of fp32 -> packed bf16 (round to nearest even)
__device__ __forceinline__ uint32_t narrow_f2(uint64_t v) {
    float lo, hi;
    unpk2(v, lo, hi);
    return pack_bf16x2_rn(lo, hi);
}

// 16-byte shared-memory store under a predicate
__device__ __forceinline__ void st_shared16_if(const void* p, const uint32_t (&v)[4], bool on) {
    asm volatile("{\n .reg .pred p;\n setp.ne.u32 p, %5, 0;\n @p st.shared.v4.u32 [%0], {%1,%2,%3,%4};\n}\n" ::"r"(smem_u32(p)),
                 "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"((uint32_t)on)
                 : "memory");
}

// 16 consecutive fp32 columns of this thread's TMEM lane into r[0..15]
#define TC_LD16(r, taddr)                                                                                      \
    asm volatile(                                                                                              \
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "                                                              \
        "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"                                      \
        : "=r"((r)[0]), "=r"((r)[1]), "=r"((r)[2]), "=r"((r)[3]), "=r"((r)[4]), "=r"((r)[5]), "=r"((r)[6]),    \
          "=r"((r)[7]), "=r"((r)[8]), "=r"((r)[9]), "=r"((r)[10]), "=r"((r)[11]), "=r"((r)[12]),              \
          "=r"((r)[13]), "=r"((r)[14]), "=r"((r)[15])                                                          \
        : "r"(taddr)                                                                                           \
        : "memory")
// 2 consecutive fp32 columns
#define TC_LD2(r, taddr) \
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : "=r"((r)[0]), "=r"((r)[1]) : "r"(taddr) : "memory")

// kFull: m == MP, every operand row belongs to a Worker (the row loops then run without branches).
template <typename T, int MP, bool kFull>
__global__ void __launch_bounds__(TcRoles<T, MP>::kThreads, 1)
gram_tc_kernel(const T* __restrict__ g, int64_t n, int m, double* __restrict__ partials, int* __restrict__ error_word) {
    using Shape = TcShape<T, MP>;
    using Smem = TcSmem<MP>;
    constexpr int RT = 2 * MP;                       // operand rows of one tile: hi rows, then lo rows
    constexpr int U = Shape::kTilesPerStage;         // tiles sharing a stage
    constexpr int kStages = Shape::kStages;
    constexpr int kChain = Shape::kChainStages;      // stages accumulated in TMEM between drains
    constexpr uint32_t kTmemCols = 512;              // kTcAccBufs buffers of kTcAccStride columns fit: all of TMEM
    static_assert(U * RT == 128, "a stage is 128 operand rows");
    static_assert((kTcAccBufs - 1) * kTcAccStride + kTcStageRows <= 512, "accumulators fit in TMEM");
    static_assert(Smem::kStages == kStages, "ring size");

    extern __shared__ unsigned char smem_raw[];
    Smem& sm = *reinterpret_cast<Smem*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    volatile int* abort = &sm.abort;
    // Roles by warp: 3 and 9 = MMA issue (on different schedulers), 4..7 = drain (TMEM quadrant = warp - 4 =
    // warp % 4), the rest = producers.
    using Roles = TcRoles<T, MP>;
    constexpr int kMmaWarp = Roles::kMmaWarp, kMmaWarpB = Roles::kMmaWarpB, kDrainWarp0 = Roles::kDrainWarp0;
    constexpr int kTcThreads = Roles::kThreads;
    const bool is_drain = warp >= kDrainWarp0 && warp < kDrainWarp0 + 4;
    const bool is_mma = warp == kMmaWarp || warp == kMmaWarpB;

    // Runs of kRun stages (a stage is U * 64 consecutive columns) are dealt round-robin to the CTAs; columns
    // past n read as zero, so a last run that sticks out past the end only adds zeros.
    constexpr int kRun = Shape::kRun;
    const int64_t nruns_all = (n + (int64_t)Shape::kStageCols * kRun - 1) / ((int64_t)Shape::kStageCols * kRun);
    const int my_stages = blockIdx.x < nruns_all ? (int)((nruns_all - blockIdx.x + gridDim.x - 1) / gridDim.x) * kRun : 0;
    const int ndrain = (my_stages + kChain - 1) / kChain;  // chains = drains

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) {
            mbar_init(&sm.full[s], Shape::kArrivals);
            for (int e = 0; e < 4; ++e) mbar_init(&sm.done[e][s], 1);
        }
        for (int b = 0; b < kTcAccBufs; ++b) {
            mbar_init(&sm.accfull[b], 1);
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
    // operand rows of Workers >= m, unused reference rows: never written by the producers, must read as zero
    for (int o = tid * 16; o < kStages * kTcStageBytes; o += kTcThreads * 16)
        *reinterpret_cast<uint4*>(&sm.stage[0][0] + o) = make_uint4(0, 0, 0, 0);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = sm.tmem_base;

    if (is_drain) {
        // ------------------------------------------------------------------ drain warps
        const int dq = warp - kDrainWarp0;  // TMEM quadrant of this warp
        // D is 128 x 144 (M = 128: row i in TMEM lane i).  Row r belongs to tile r / RT of the stage and
        // needs that tile's own columns only: D[r][cb + c] (hi columns) + D[r][cb + MP + c] (lo columns),
        // and the tile's two reference columns.
        const int row = dq * 32 + lane;
        const int tu = row / RT;
        const uint32_t lane_addr = tmem_base + ((uint32_t)(dq * 32) << 16);
        const uint32_t cb = (uint32_t)(tu * RT);
        constexpr int W = MP < 32 ? MP : 32;  // Gram columns per round of loads
        uint64_t facc[MP / 2];                // packed pairs of fp32 sums
        float ft = 0.f;
#pragma unroll
        for (int e = 0; e < MP / 2; ++e) facc[e] = 0ull;
#pragma unroll 4
        for (int e = 0; e < MP; ++e) sm.acc64[e * 128 + row] = 0.0;
        sm.t64[row] = 0.0;
        int b = 0, since_wide = 0;
        uint32_t full_par = 0;
        for (int f = 0; f < ndrain; ++f) {
            mbar_wait(&sm.accfull[b], full_par, abort);  // the chain's MMAs have completed
            __syncwarp();
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint32_t acc_addr = lane_addr + (uint32_t)(b * kTcAccStride);
            uint32_t tv[2];
#pragma unroll
            for (int c0 = 0; c0 < MP; c0 += W) {
                uint32_t v[W], w[W];
#pragma unroll
                for (int q = 0; q < W; q += 16) {
                    TC_LD16(v + q, acc_addr + cb + c0 + q);
                    TC_LD16(w + q, acc_addr + cb + MP + c0 + q);
                }
                if (c0 == 0) TC_LD2(tv, acc_addr + 128 + 2 * tu);
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
                for (int jj = 0; jj < W / 2; ++jj)
                    facc[c0 / 2 + jj] = add2(facc[c0 / 2 + jj], add2(pk2(v[2 * jj], v[2 * jj + 1]), pk2(w[2 * jj], w[2 * jj + 1])));
            }
            ft += __uint_as_float(tv[0]) + __uint_as_float(tv[1]);
            // the accumulator buffer is free again as soon as every drain warp has read it
            asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
            __syncwarp();
            if (lane == 0) mbar_arrive(&sm.accempty[b]);
            if (++b == kTcAccBufs) {
                b = 0;
                full_par ^= 1u;
            }
            if (++since_wide == kTcWideEvery || f == ndrain - 1) {
                since_wide = 0;
#pragma unroll
                for (int e = 0; e < MP / 2; ++e) {
                    float lo, hi;
                    unpk2(facc[e], lo, hi);
                    sm.acc64[(2 * e) * 128 + row] += (double)lo;
                    sm.acc64[(2 * e + 1) * 128 + row] += (double)hi;
                    facc[e] = 0ull;
                }
                sm.t64[row] += (double)ft;
                ft = 0.f;
            }
        }
    } else if (is_mma) {
        // ------------------------------------------------------------------ MMA issue
        // The issuing thread runs in step with the tensor pipe (an MMA is accepted about when the one before it
        // completes), so the time it spends on barrier waits is time the pipe idles.  Two warps therefore issue,
        // taking the groups of stages alternately: one warp's waits overlap the other's MMAs.  The groups use
        // different stages and different accumulator buffers, so the two instruction streams need no order.
        if (lane == 0) {
            // kind::f16, fp32 accumulate, bf16 x bf16, both K-major, N = 144, M = 128
            const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTcStageRows >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
            const uint64_t desc0 = tc_smem_desc(smem_u32(sm.stage[0]));
            for (int c = warp == kMmaWarp ? 0 : 1; c < ndrain; c += kTcMmaWarps) {
                const int b = c % kTcAccBufs;
                mbar_wait<false>(&sm.accempty[b], (uint32_t)(((c / kTcAccBufs) & 1) ^ 1), abort);
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t d_tmem = tmem_base + (uint32_t)(b * kTcAccStride);
#pragma unroll
                for (int t = 0; t < kChain; ++t) {
                    const int p = c * kChain + t;
                    if (p < my_stages) {
                        const int s = p % kStages, rev = p / kStages;
                        mbar_wait<false>(&sm.full[s], (uint32_t)(rev & 1), abort);
                        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                        // the start-address field counts 16-byte units; a K step of 16 bf16 is 32 bytes
                        const uint64_t desc = desc0 + (uint64_t)(s * (kTcStageBytes >> 4));
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const uint32_t accumulate = (t == 0 && k == 0) ? 0u : 1u;
                            asm volatile(
                                "{\n .reg .pred p;\n setp.ne.u32 p, %4, 0;\n"
                                "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n" ::"r"(d_tmem),
                                "l"(desc + 2 * k), "l"(desc + 2 * k), "r"(idesc), "r"(accumulate)
                                : "memory");
                        }
                        // the release group's stages are free once these MMAs have completed
                        if (t % kTcRelease == kTcRelease - 1 || p == my_stages - 1)
                            asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                                             smem_u32(&sm.done[rev & 3][s / kTcRelease]))
                                         : "memory");
                    }
                }
                // the chain's accumulator is complete once all of its MMAs have completed
                asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                                 smem_u32(&sm.accfull[b]))
                             : "memory");
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ producer warps
        constexpr int RPL = Shape::kRowsPerLane;     // Workers per lane
        constexpr int CPI = Shape::kChunksPerItem;   // 8-column chunks per item = lanes per row group
        constexpr int NW = 16 / RPL * 4;             // 32-bit registers per chunk: 4 (bf16) or 8 (fp32)
        constexpr int SPI = Shape::kStagesPerItem, IPS = Shape::kItemsPerStage;
        constexpr int kTeam = Shape::kTeam, kTeams = Shape::kTeams;
        constexpr int kStageChunks = Shape::kStageCols / 8;
        constexpr bool kBf16 = sizeof(T) == 2;
        // a warp prefetches the item this many of its own items ahead into L2 (measured: helps bf16 storage a
        // little, costs fp32 storage more than it brings)
        constexpr int kTcPrefetchAhead = kBf16 ? QN_TC_PREFETCH_BF16 : QN_TC_PREFETCH_F32;
        const int pw = Roles::producer_index(warp);
        const int team = pw / kTeam, half = pw % kTeam;
        const int rq = lane / CPI, cl = lane % CPI;
        const int w0 = half * Shape::kRowsPerWarp + rq * RPL;  // first Worker of this lane's rows
        const int my_items = my_stages / SPI * IPS;  // my_stages is a multiple of kRun, kRun of SPI
        uint32_t raw[RPL][NW];

        // first stage of item k (an item is SPI whole stages or one of the IPS column parts of a stage)
        auto item_stage = [&](int k) -> int { return k / IPS * SPI; };
        // first column of the CTA's p-th stage
        auto stage_col0 = [&](int p) -> int64_t {
            return ((blockIdx.x + (int64_t)(p / kRun) * gridDim.x) * kRun + p % kRun) * Shape::kStageCols;
        };
        // first column of item k (the stages of an item are adjacent in memory: they belong to one run)
        auto item_col0 = [&](int k) -> int64_t { return stage_col0(item_stage(k)) + (k % IPS) * Shape::kItemCols; };
        // first column of this lane's chunk in item k, or -1 if the item or the chunk lies past the end
        auto item_col = [&](int k) -> int64_t {
            if (k >= my_items) return -1;
            const int64_t c = item_col0(k) + cl * 8;
            // rows are 32-byte aligned and n is a multiple of 8 on this path (see qn_gram_tc_applicable),
            // so an 8-column chunk is never cut by the end of the row
            return c < n ? c : -1;
        };
        // Predicated load (no branch): the registers read as zero for a chunk past the end or a row without a Worker.
        auto load_row = [&](int j, int64_t col) {
            const bool on = col >= 0 && (kFull || w0 + j < m);
            const T* p = g + (on ? (int64_t)(w0 + j) * n + col : 0);
            if (kBf16)
                asm volatile(
                    "{\n .reg .pred p;\n setp.ne.u32 p, %5, 0;\n mov.u32 %0, 0;\n mov.u32 %1, 0;\n mov.u32 %2, 0;\n mov.u32 %3, 0;\n"
                    "@p ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];\n}\n"
                    : "=&r"(raw[j][0]), "=&r"(raw[j][1]), "=&r"(raw[j][2]), "=&r"(raw[j][3])
                    : "l"(p), "r"((uint32_t)on));
            else
                asm volatile(
                    "{\n .reg .pred p;\n setp.ne.u32 p, %9, 0;\n mov.u32 %0, 0;\n mov.u32 %1, 0;\n mov.u32 %2, 0;\n mov.u32 %3, 0;\n"
                    "mov.u32 %4, 0;\n mov.u32 %5, 0;\n mov.u32 %6, 0;\n mov.u32 %7, 0;\n"
                    "@p ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];\n}\n"
                    : "=&r"(raw[j][0]), "=&r"(raw[j][1]), "=&r"(raw[j][2]), "=&r"(raw[j][3]), "=&r"(raw[j][NW - 4]),
                      "=&r"(raw[j][NW - 3]), "=&r"(raw[j][NW - 2]), "=&r"(raw[j][NW - 1])
                    : "l"(p), "r"((uint32_t)on));
        };
        // Plain load for items that lie wholly inside the rows (every item but a CTA's last few).
        auto load_row_plain = [&](int j, const T* p) {
            if (kBf16)
                asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                             : "=r"(raw[j][0]), "=r"(raw[j][1]), "=r"(raw[j][2]), "=r"(raw[j][3])
                             : "l"(p));
            else
                asm volatile("ld.global.nc.L1::no_allocate.v8.u32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
                             : "=r"(raw[j][0]), "=r"(raw[j][1]), "=r"(raw[j][2]), "=r"(raw[j][3]), "=r"(raw[j][NW - 4]),
                               "=r"(raw[j][NW - 3]), "=r"(raw[j][NW - 2]), "=r"(raw[j][NW - 1])
                             : "l"(p));
        };
        // a warp's part of an item is 64 lines of 128 bytes (its rows x 8 KB / rows): two per lane
        auto prefetch_item = [&](int k) {
            constexpr int kLinesPerRow = Shape::kItemCols * (int)sizeof(T) / 128;
            constexpr int kLineCols = 128 / (int)sizeof(T);
            if (k >= my_items) return;
            const int64_t c0 = item_col0(k);
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int q = lane + 32 * t, row = half * Shape::kRowsPerWarp + q / kLinesPerRow;
                const int64_t c = c0 + (q % kLinesPerRow) * kLineCols;
                if (row < m && c < n) asm volatile("prefetch.global.L2 [%0];" ::"l"(g + (int64_t)row * n + c));
            }
        };

        if (kTcPrefetchAhead > 1) prefetch_item(team + kTeams);
        {
            const int64_t col = item_col(team);
#pragma unroll
            for (int j = 0; j < RPL; ++j) load_row(j, col);
        }
        const float inv_m = 1.0f / (float)m;
        int xpar = 0;  // buffer of the team's exchange area used by this item
        for (int k = team; k < my_items; k += kTeams) {
            // the lane's chunk: its stage, its tile in the stage and its 16-byte slot in the tile's 128-byte rows
            const int ch_item = (k % IPS) * CPI + cl;                  // chunk index counted from the item's first stage
            const int p = item_stage(k) + ch_item / kStageChunks;      // stage use the chunk belongs to
            const int s = p % kStages;
            const int ch = ch_item % kStageChunks;
            const int tu = ch >> 3, c8 = ch & 7;
            unsigned char* rows = sm.stage[s] + (tu * RT + w0) * 128;  // operand row of hi(Worker w0)
            const uint32_t xo = (uint32_t)c8 << 4;
            const int64_t col_next = item_col(k + kTeams);
            // warp-uniform: the whole next item lies inside the rows (then no load needs a predicate)
            const bool next_inside = (kBf16 || QN_TC_FASTPATH_F32) && kFull && k + kTeams < my_items && item_col0(k + kTeams) + Shape::kItemCols <= n;
            const T* next_base = g + (int64_t)w0 * n + (next_inside ? col_next : 0);
            if (kTcPrefetchAhead > 0) prefetch_item(k + kTcPrefetchAhead * kTeams);

            // ---- the reference of the lane's 8 columns (identical in all lanes and warps that share them)
            uint32_t rb[4];   // bf16 storage: r as four packed pairs; fp32 storage: rh (hi part of r)
            uint32_t rlo[4];  // fp32 storage: rl
            uint64_t rf[4];   // fp32 storage: r = rh + rl as pairs of fp32
            if (kBf16) {
                uint32_t sum[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    uint32_t t[RPL];
#pragma unroll
                    for (int j = 0; j < RPL; ++j) t[j] = raw[j][e];
#pragma unroll
                    for (int span = RPL / 2; span > 0; span >>= 1) {
#pragma unroll
                        for (int j = 0; j < span; ++j) t[j] = add_bf2(t[2 * j], t[2 * j + 1]);
                    }
                    sum[e] = t[0];
#pragma unroll
                    for (int o = CPI; o < 32; o <<= 1) sum[e] = add_bf2(sum[e], __shfl_xor_sync(0xffffffffu, sum[e], o));
                }
                if (kTeam == 2) {
                    // the other warp of the team holds the other 32 rows of these columns
                    uint4* xb = &sm.xbuf[team][xpar][0][0][0];
                    if (rq == 0) xb[(half * 16 + cl) * 2] = make_uint4(sum[0], sum[1], sum[2], sum[3]);
                    asm volatile("bar.sync %0, 64;" ::"r"(1 + team) : "memory");
                    const uint4 o = xb[((half ^ 1) * 16 + cl) * 2];
                    sum[0] = add_bf2(sum[0], o.x);
                    sum[1] = add_bf2(sum[1], o.y);
                    sum[2] = add_bf2(sum[2], o.z);
                    sum[3] = add_bf2(sum[3], o.w);
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) rb[e] = mul_bf2(sum[e], pack_bf16x2_rn(inv_m, inv_m));
            } else {
                uint64_t sum[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    sum[e] = pk2(raw[0][2 * e], raw[0][2 * e + 1]);
#pragma unroll
                    for (int j = 1; j < RPL; ++j) sum[e] = add2(sum[e], pk2(raw[j][2 * e], raw[j][2 * e + 1]));
#pragma unroll
                    for (int o = CPI; o < 32; o <<= 1)
                        sum[e] = add2(sum[e], (uint64_t)__shfl_xor_sync(0xffffffffu, (unsigned long long)sum[e], o));
                }
                if (kTeam == 2) {
                    uint4* xb = &sm.xbuf[team][xpar][0][0][0];
                    if (rq == 0) {
                        xb[(half * 16 + cl) * 2] = make_uint4((uint32_t)sum[0], (uint32_t)(sum[0] >> 32), (uint32_t)sum[1], (uint32_t)(sum[1] >> 32));
                        xb[(half * 16 + cl) * 2 + 1] = make_uint4((uint32_t)sum[2], (uint32_t)(sum[2] >> 32), (uint32_t)sum[3], (uint32_t)(sum[3] >> 32));
                    }
                    asm volatile("bar.sync %0, 64;" ::"r"(1 + team) : "memory");
                    const uint4 o0 = xb[((half ^ 1) * 16 + cl) * 2], o1 = xb[((half ^ 1) * 16 + cl) * 2 + 1];
                    sum[0] = add2(sum[0], pk2(o0.x, o0.y));
                    sum[1] = add2(sum[1], pk2(o0.z, o0.w));
                    sum[2] = add2(sum[2], pk2(o1.x, o1.y));
                    sum[3] = add2(sum[3], pk2(o1.z, o1.w));
                }
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const uint64_t mean = mul2(sum[e], pk2(__float_as_uint(inv_m), __float_as_uint(inv_m)));
                    // the reference is the mean rounded to 16 significant bits, so that rh + rl is r exactly
                    rb[e] = narrow_f2(mean);
                    const uint64_t rhf = widen_bf2(rb[e]);
                    rlo[e] = narrow_f2(sub2(mean, rhf));
                    rf[e] = add2(rhf, widen_bf2(rlo[e]));
                }
            }
            xpar ^= 1;

            // the stage must have been consumed by the MMAs of its previous use (revolution rev - 1 of the ring);
            // the stages of one item belong to the same release group
            const int rev = p / kStages;
            if (rev > 0) mbar_wait(&sm.done[(rev - 1) & 3][s / kTcRelease], (uint32_t)((rev - 1) >> 2) & 1u, abort);
            if (rq == 0 && half == 0) {
                // reference rows 128 + 2 tu (rh) and 129 + 2 tu (rl; zero and never written for bf16 storage)
                unsigned char* rr = sm.stage[s] + (128 + 2 * tu) * 128;
                *reinterpret_cast<uint4*>(rr + (xo ^ (uint32_t)((2 * tu) << 4))) = make_uint4(rb[0], rb[1], rb[2], rb[3]);
                if (!kBf16)
                    *reinterpret_cast<uint4*>(rr + 128 + (xo ^ (uint32_t)((2 * tu + 1) << 4))) =
                        make_uint4(rlo[0], rlo[1], rlo[2], rlo[3]);
            }

            // the row loop, compiled twice: with plain loads of the next item (the common case) and with
            // predicated ones (the next item is cut by the end of the rows, does not exist, or m < MP)
            auto convert_rows = [&](auto plain_tag) {
                constexpr bool kPlain = decltype(plain_tag)::value;
#pragma unroll
            for (int j = 0; j < RPL; ++j) {
                {
                    uint32_t hw[4], lw[4];
#pragma unroll
                    for (int e = 0; e < 4; ++e) {
                        if (kBf16) {
                            // TwoSum of a = g and b = -r: hw = fl(a + b), lw = (a + b) - hw exactly
                            const uint32_t a = raw[j][e], r = rb[e];
                            const uint32_t sum = sub_bf2(a, r);
                            const uint32_t av = add_bf2(sum, r);          // a' = s - b
                            const uint32_t bv = sub_bf2(sum, av);         // b' = s - a'
                            const uint32_t da = sub_bf2(a, av);           // a - a'
                            hw[e] = sum;
                            lw[e] = sub_bf2(da, add_bf2(r, bv));          // (a - a') + (b - b')
                        } else {
                            const uint64_t x = sub2(pk2(raw[j][2 * e], raw[j][2 * e + 1]), rf[e]);
                            hw[e] = narrow_f2(x);
                            lw[e] = narrow_f2(sub2(x, widen_bf2(hw[e])));
                        }
                    }
                    // this row's registers are free: fetch the same lane's row of the warp's next item into them
                    if (kPlain)
                        load_row_plain(j, next_base + (int64_t)j * n);
                    else
                        load_row(j, col_next);
                    // operand row w0 + j of the tile; (w0 + j) & 7 == j & 7
                    const uint32_t off = (uint32_t)(j * 128) + (xo ^ (uint32_t)((j & 7) << 4));
                    if (kFull) {
                        *reinterpret_cast<uint4*>(rows + off) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                        *reinterpret_cast<uint4*>(rows + MP * 128 + off) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
                    } else {
                        // rows without a Worker stay zero: predicated stores keep the row loop free of branches
                        st_shared16_if(rows + off, hw, w0 + j < m);
                        st_shared16_if(rows + MP * 128 + off, lw, w0 + j < m);
                    }
                }
            }
            };
            if (next_inside)
                convert_rows(std::true_type{});
            else
                convert_rows(std::false_type{});
            // make the generic-proxy stores visible to the tensor core, then hand the warp's part of the item over
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            __syncwarp();
            if (lane == 0) {
#pragma unroll
                for (int q = 0; q < SPI; ++q) mbar_arrive(&sm.full[(item_stage(k) + q) % kStages]);
            }
        }
    }

    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    const double qnan = __longlong_as_double(0x7ff8000000000000ll);
    const bool poisoned = *abort != 0;
    double* out = partials + (int64_t)blockIdx.x * qn_partial_len(m);
    const int tri = m * (m + 1) / 2;
    if (tid < 128) {
        // acc64[bc][row]: D rows u*RT + a (hi part of Worker a in tile u) and u*RT + MP + a (lo part), already
        // folded over the hi and lo columns of Worker bc
        constexpr int PER = MP * MP / 128;
        const int a = tid % MP, h = tid / MP;
#pragma unroll 4
        for (int e = 0; e < PER; ++e) {
            const int bc = h * PER + e;
            if (a <= bc && bc < m) {
                double v = 0.0;
#pragma unroll
                for (int u = 0; u < U; ++u) v += sm.acc64[bc * 128 + u * RT + a] + sm.acc64[bc * 128 + u * RT + MP + a];
                out[qn_tri_index(m, a, bc)] = poisoned ? qnan : v;
            }
        }
    } else if (tid - 128 < m) {
        const int a = tid - 128;
        double v = 0.0;
#pragma unroll
        for (int u = 0; u < U; ++u) v += sm.t64[u * RT + a] + sm.t64[u * RT + MP + a];
        out[tri + a] = poisoned ? qnan : v;
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
    auto kern = m == MP ? gram_tc_kernel<T, MP, true> : gram_tc_kernel<T, MP, false>;
    const size_t smem = sizeof(TcSmem<MP>) + 1024;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, TcRoles<T, MP>::kThreads, smem, st>>>(g, n, m, partials, error_word);
    return cudaGetLastError();
}

template <typename T>
static cudaError_t launch_tc_any(const T* g, int64_t n, int m, double* partials, int* num_partials, int max_partials,
                                 int* error_word, cudaStream_t st) {
    const int mp = m <= 16 ? 16 : m <= 32 ? 32 : 64;
    const int64_t stage_cols = 64 * (64 / mp);
    const int64_t stage_row_bytes = stage_cols * (int64_t)sizeof(T);
    const int64_t run_cols = stage_cols * (stage_row_bytes >= kTcRunBytes ? 1 : kTcRunBytes / stage_row_bytes);
    const int64_t nruns = (n + run_cols - 1) / run_cols;
    const int sms = qn_sm_count();
    int grid = (int)(nruns < sms ? nruns : sms);
    if (grid > max_partials) grid = max_partials;
    *num_partials = grid;
    if (mp == 16) return launch_tc<T, 16>(g, n, m, partials, grid, error_word, st);
    if (mp == 32) return launch_tc<T, 32>(g, n, m, partials, grid, error_word, st);
    return launch_tc<T, 64>(g, n, m, partials, grid, error_word, st);
}

template <typename T, int MP>
static cudaError_t preload_tc() {
    const size_t smem = sizeof(TcSmem<MP>) + 1024;
    cudaFuncAttributes a;
    cudaError_t e = cudaFuncGetAttributes(&a, gram_tc_kernel<T, MP, true>);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gram_tc_kernel<T, MP, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e == cudaSuccess) e = cudaFuncGetAttributes(&a, gram_tc_kernel<T, MP, false>);
    if (e == cudaSuccess) e = cudaFuncSetAttribute(gram_tc_kernel<T, MP, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    return e;
}

}  // namespace qn

cudaError_t qn_gram_tc_preload() {
    cudaError_t e = qn::preload_tc<float, 16>();
    if (e == cudaSuccess) e = qn::preload_tc<float, 32>();
    if (e == cudaSuccess) e = qn::preload_tc<float, 64>();
    if (e == cudaSuccess) e = qn::preload_tc<__nv_bfloat16, 16>();
    if (e == cudaSuccess) e = qn::preload_tc<__nv_bfloat16, 32>();
    if (e == cudaSuccess) e = qn::preload_tc<__nv_bfloat16, 64>();
    return e;
}

bool qn_gram_tc_applicable(qn_dtype dtype, const void* g, int64_t n, int m) {
    const int64_t elem = dtype == QN_F32 ? 4 : 2;
    // every 8-column chunk of a row is fetched with one load: 16 bytes (bf16) or 32 bytes (fp32), aligned
    const int64_t chunk = 8 * elem;
    return m > 8 && m <= QN_MAX_M && n >= QN_TC_MIN_N && (reinterpret_cast<uintptr_t>(g) % chunk == 0) &&
           (n % 8 == 0);
}

cudaError_t qn_launch_gram_tc(qn_dtype dtype, const void* g, int64_t n, int m, double* partials, int* num_partials,
                              int max_partials, int* error_word, cudaStream_t st) {
    if (dtype == QN_F32)
        return qn::launch_tc_any(static_cast<const float*>(g), n, m, partials, num_partials, max_partials, error_word, st);
    return qn::launch_tc_any(static_cast<const __nv_bfloat16*>(g), n, m, partials, num_partials, max_partials,
                             error_word, st);
}
