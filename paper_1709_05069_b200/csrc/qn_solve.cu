// Single-CTA kernel between the two streaming passes: deterministic sum of the Gram partials, exact
// m x m centring, two-sided Jacobi eigen-decomposition of G^T G in fp64, sigma_k, the lambda cut-off j
// and the coefficient vector of the final combination.
//
// Paper, Section 2: V_G and Sigma_G come from the eigenpairs of G^H G; j is fixed by
// sigma_j >= lambda sigma_1 > sigma_{j+1}; Eq. (4) with z = gbar needs alpha_k = gbar^T u_k and
// alpha_k sigma_k^-1 y_k.  With w = G^T gbar one has alpha_k = v_k^T w / sigma_k, and both sums of
// Eq. (4) collapse onto one m-vector d = sum_{k<=j} v_k (v_k^T w) / sigma_k^2:
//     sum alpha_k u_k = G d,   sum alpha_k sigma_k^-1 y_k = Theta d.
//
// Centring: the streaming pass shifts each column by a reference r_i that only approximates the
// mean.  With x' = g - r, C' = sum x' x'^T, t = sum x' r and P = I - 11^T/m:
//     G^T G = P C' P,      G^T gbar = P t + P C' 1 / m,
// exactly, for any r (r = 0 gives the raw Gram of the asynchronous window).
#include "qn_device.cuh"

namespace qn {

constexpr int kLd = QN_MAX_M + 2;  // leading dimension of the shared matrices (even: 2x1 pairs of doubles are 16-byte aligned)
constexpr int kMaxSweeps = 30;

struct SolveSmem {
    double A[QN_MAX_M * kLd];
    double V[QN_MAX_M * kLd];  // also scratch for the partial sums before the Jacobi phase
    double A2[QN_MAX_M * kLd], V2[QN_MAX_M * kLd];  // the Jacobi rounds read one copy and write the other
    union {
        double B[QN_MAX_M * kLd];  // reference-shifted Gram of theta (learning-rate cap only; built after the fp32 phase)
        struct {
            float A[2][QN_MAX_M * kLd], V[2][QN_MAX_M * kLd];  // fp32 pre-diagonalisation: A / ||A||_F and its rotations
            float rot_c[QN_MAX_M / 2], rot_s[QN_MAX_M / 2];
        } f;
    };
    double w[QN_MAX_M];
    double rowsum[QN_MAX_M];
    double mu[QN_MAX_M];
    double sigma[QN_MAX_M];
    double rot_c[QN_MAX_M / 2], rot_s[QN_MAX_M / 2];
    double modec[QN_MAX_M];
    double d[QN_MAX_M];
    double red[32];
    double diag_scale;  // largest diagonal entry of the uncentred Gram
    int order[QN_MAX_M];
    int flag_nonfinite;
    int flag_rotated;
    int flag_timeout;
    int j;
    double tau_eff;
};

__device__ __forceinline__ double block_sum(double x, double* red) {
    // fixed-order block reduction; every thread returns the total
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
    x = warp_sum(x);
    __syncthreads();
    if (lane == 0) red[warp] = x;
    __syncthreads();
    double s = 0.0;
    for (int i = 0; i < nw; ++i) s += red[i];
    return s;
}

// Where physical position i of the tournament table goes after a round: position 0 stays, the other top positions
// 2k move right, the bottom positions 2k+1 move left, the ends turn round.
__device__ __forceinline__ int next_pos(int i, int M2) {
    if (M2 == 2 || i == 0) return i;
    if (i == 1) return 2;
    if (i & 1) return i - 2;
    return i == M2 - 2 ? M2 - 1 : i + 2;
}

// Pre-diagonalisation in fp32: the same systolic round-robin Jacobi as the fp64 phase of the kernel, on A / ||A||_F.
// Vector fp64 runs at an eighth of the fp32 rate on this part and bounds the fp64 rounds from m = 32 on; the fp32
// rounds cost a fraction.  The result is only an approximation (V orthogonal and V^T A V diagonal to about 1e-6):
// the kernel then re-orthonormalises V in fp64, transforms A with it and lets the fp64 Jacobi finish from there
// in two or three sweeps.  Returns the buffer index (0 or 1) that holds the final V.
#ifndef QN_SOLVE_PRE_MIN_M
#define QN_SOLVE_PRE_MIN_M 12
#endif
constexpr int kPreMinM = QN_SOLVE_PRE_MIN_M;  // below this the fp64 sweeps are short anyway
#ifndef QN_SOLVE_PRE_SWEEPS
#define QN_SOLVE_PRE_SWEEPS 8
#endif
constexpr int kPreMaxSweeps = QN_SOLVE_PRE_SWEEPS;
// largest off-diagonal entry (relative to ||A||_F) at which the fp32 sweeps stop.  Measured totals of the kernel in
// thousands of cycles at m = 16 / 32 / 64: 3e-6: 164 / 330 / 1287, 3e-5: 163 / 335 / 1343, 3e-4: 152 / 354 / 1414,
// 3e-3: 159 / 374 / 1621 (a looser stop saves fp32 sweeps and costs more fp64 sweeps, which are 1.6 times as long).
#ifndef QN_SOLVE_PRE_THR
#define QN_SOLVE_PRE_THR 3e-6f
#endif
__device__ __forceinline__ int jacobi_fp32(SolveSmem& sm, int M2, int tid, int jthreads) {
    const int H = M2 / 2, N = M2 - 1;
    const int pa_idx = tid / H, pb_idx = tid % H;
    const bool worker = tid < H * H;
    const int ra = 2 * pa_idx, cb = 2 * pb_idx;
    const int nr0 = next_pos(ra, M2), nr1 = next_pos(ra + 1, M2), nc0 = next_pos(cb, M2), nc1 = next_pos(cb + 1, M2);
    const float thr_rot = 1e-9f, thr_done = QN_SOLVE_PRE_THR;  // entries are relative to ||A||_F = 1
    int cur = 0;
    for (int sweep = 0; sweep < kPreMaxSweeps; ++sweep) {
        for (int r = 0; r < N; ++r) {
            const float* Ar = sm.f.A[cur];
            const float* Vr = sm.f.V[cur];
            float* Aw = sm.f.A[cur ^ 1];
            float* Vw = sm.f.V[cur ^ 1];
            float x00 = 0.f, x01 = 0.f, x10 = 0.f, x11 = 0.f;
            if (worker) {
                const float2 r0 = *reinterpret_cast<const float2*>(&Ar[ra * kLd + cb]);
                const float2 r1 = *reinterpret_cast<const float2*>(&Ar[(ra + 1) * kLd + cb]);
                x00 = r0.x;
                x01 = r0.y;
                x10 = r1.x;
                x11 = r1.y;
                if (pa_idx == pb_idx) {
                    float c = 1.f, sn = 0.f;
                    if (fabsf(x01) > thr_rot) {
                        const float df = x11 - x00, of = x01 + x01;
                        const float r2 = fmaf(df, df, of * of);
                        const float h = r2 * rsqrtf(r2);
                        const float tf = copysignf(__fdividef(fabsf(of), fabsf(df) + h), df * of);
                        c = rsqrtf(fmaf(tf, tf, 1.0f));
                        sn = tf * c;
                    }
                    sm.f.rot_c[pa_idx] = c;
                    sm.f.rot_s[pa_idx] = sn;
                }
            }
            asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
            if (worker) {
                const float ca = sm.f.rot_c[pa_idx], sa = sm.f.rot_s[pa_idx];
                const float cbr = sm.f.rot_c[pb_idx], sbr = sm.f.rot_s[pb_idx];
                const float2 v0 = *reinterpret_cast<const float2*>(&Vr[ra * kLd + cb]);
                const float2 v1 = *reinterpret_cast<const float2*>(&Vr[(ra + 1) * kLd + cb]);
                const float t00 = cbr * x00 - sbr * x01, t01 = sbr * x00 + cbr * x01;
                const float t10 = cbr * x10 - sbr * x11, t11 = sbr * x10 + cbr * x11;
                float y00 = ca * t00 - sa * t10, y10 = sa * t00 + ca * t10;
                float y01 = ca * t01 - sa * t11, y11 = sa * t01 + ca * t11;
                if (pa_idx == pb_idx) y01 = y10 = 0.5f * (y01 + y10);
                Aw[nr0 * kLd + nc0] = y00;
                Aw[nr0 * kLd + nc1] = y01;
                Aw[nr1 * kLd + nc0] = y10;
                Aw[nr1 * kLd + nc1] = y11;
                Vw[ra * kLd + nc0] = cbr * v0.x - sbr * v0.y;
                Vw[ra * kLd + nc1] = sbr * v0.x + cbr * v0.y;
                Vw[(ra + 1) * kLd + nc0] = cbr * v1.x - sbr * v1.y;
                Vw[(ra + 1) * kLd + nc1] = sbr * v1.x + cbr * v1.y;
            }
            asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
            cur ^= 1;
        }
        int big = 0;
        for (int e = tid; e < M2 * M2; e += jthreads) {
            const int k = e / M2, l = e % M2;
            big |= (k != l) && (fabsf(sm.f.A[cur][k * kLd + l]) > thr_done);
        }
        big = __any_sync(0xffffffffu, big);
        if (big && (tid & 31) == 0) sm.flag_rotated = 1;
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
        const int rotated = sm.flag_rotated;
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
        if (tid == 0) sm.flag_rotated = 0;
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
        if (!rotated) break;
    }
    return cur;
}

__global__ void __launch_bounds__(1024, 1) solve_kernel(qn_solve_params prm) {
    extern __shared__ __align__(16) unsigned char smem_raw[];
    SolveSmem& sm = *reinterpret_cast<SolveSmem*>(smem_raw);
    const int m = prm.m;
    const int tid = threadIdx.x, nthr = blockDim.x;
    const int tri_len = m * (m + 1) / 2;
    // the second solve of a step whose Gram pass was repeated in fp64: nothing to do unless the first one asked for it
    if (prm.only_if_redo && (prm.result->redo & 1) == 0) return;

    if (tid == 0) {
        sm.flag_nonfinite = 0;
        sm.flag_rotated = 0;
        sm.j = 0;
        sm.flag_timeout = 0;
        if (prm.error_word && *prm.error_word) {  // a streaming kernel gave up on a wait: report and clear
            sm.flag_timeout = 1;
            *prm.error_word = 0;
        }
    }
    // ---------------------------------------------------------------- phase 1: C' and t
    if (prm.source == QN_SRC_PARTIALS) {
        const int E = tri_len + m;
        double* packed = sm.V;  // E <= 2144 doubles fits in V (4160)
        for (int e = tid; e < E; e += nthr) {
            double s0 = 0, s1 = 0, s2 = 0, s3 = 0;
            int p = 0;
            for (; p + 3 < prm.num_partials; p += 4) {
                s0 += prm.partials[(int64_t)(p + 0) * E + e];
                s1 += prm.partials[(int64_t)(p + 1) * E + e];
                s2 += prm.partials[(int64_t)(p + 2) * E + e];
                s3 += prm.partials[(int64_t)(p + 3) * E + e];
            }
            for (; p < prm.num_partials; ++p) s0 += prm.partials[(int64_t)p * E + e];
            packed[e] = (s0 + s1) + (s2 + s3);
        }
        __syncthreads();
        for (int e = tid; e < m * m; e += nthr) {
            const int k = e / m, l = e % m;
            sm.A[k * kLd + l] = packed[k <= l ? qn_tri_index(m, k, l) : qn_tri_index(m, l, k)];
        }
        if (tid < m) sm.w[tid] = packed[tri_len + tid];
        __syncthreads();
        if (prm.raw_gram)
            for (int e = tid; e < m * m; e += nthr) prm.raw_gram[e] = sm.A[(e / m) * kLd + (e % m)];
    } else {
        // QN_SRC_WINDOW: the raw Gram (w follows from it in the centring below); QN_SRC_SUMMED: a centred Gram
        // followed by w, e.g. the sum over column shards of what qn_gram wrote (the centring below leaves an
        // already centred pair unchanged up to rounding: P (P C P) P = P C P and 1^T w = 0)
        for (int e = tid; e < m * m; e += nthr) sm.A[(e / m) * kLd + (e % m)] = prm.raw_gram[e];
        if (tid < m) sm.w[tid] = prm.source == QN_SRC_SUMMED ? prm.raw_gram[m * m + tid] : 0.0;
        __syncthreads();
    }

    // ---------------------------------------------------------------- phase 2: exact centring
    if (tid < m) {
        double s = 0.0;
        for (int l = 0; l < m; ++l) s += sm.A[tid * kLd + l];
        sm.rowsum[tid] = s;
    }
    __syncthreads();
    double tot = 0.0, tsum = 0.0, dmax = 0.0;
    for (int k = 0; k < m; ++k) {
        tot += sm.rowsum[k];
        tsum += sm.w[k];
        dmax = fmax(dmax, sm.A[k * kLd + k]);
    }
    if (tid == 0) sm.diag_scale = dmax;
    const double inv_m = 1.0 / (double)m;
    __syncthreads();
    bool bad = false;
    for (int e = tid; e < m * m; e += nthr) {
        const int k = e / m, l = e % m;
        const double c = sm.A[k * kLd + l] - (sm.rowsum[k] + sm.rowsum[l]) * inv_m + tot * inv_m * inv_m;
        sm.A[k * kLd + l] = c;
        bad |= !isfinite(c);
        if (prm.gram_out) prm.gram_out[e] = c;
    }
    if (tid < m) {
        double wk = sm.w[tid] - tsum * inv_m + sm.rowsum[tid] * inv_m - tot * inv_m * inv_m;
        if (prm.rhs_raw) {
            // coefficients for an arbitrary z: G^T z = P (g_k^T z)_k, because the centring removes the same
            // gbar^T z from every entry
            double rs = 0.0;
            for (int l = 0; l < m; ++l) rs += prm.rhs_raw[l];
            wk = prm.rhs_raw[tid] - rs * inv_m;
        }
        bad |= !isfinite(wk);
        // every thread has read w (tsum) before the barrier above; only thread tid rewrites w[tid]
        sm.w[tid] = wk;
        if (prm.gram_out) prm.gram_out[m * m + tid] = wk;
    }
    if (bad) sm.flag_nonfinite = 1;
    __syncthreads();
    if (prm.gram_only) {
        if (tid == 0 && prm.result) {
            prm.result->status = sm.flag_timeout ? QN_ERR_DEVICE_TIMEOUT : sm.flag_nonfinite ? QN_ERR_NONFINITE : QN_OK;
            prm.result->j = 0;
            prm.result->sweeps = 0;
            prm.result->redo = 0;
        }
        return;
    }
    if (sm.flag_nonfinite) {  // the SGD update: no mode kept
        if (tid < QN_MAX_M) {
            prm.coef->c[tid] = 0.f;
            prm.result->sigma[tid] = 0.0;
        }
        if (tid == 0) {
            prm.coef->tau = (float)prm.tau;
            prm.coef->inv_m = (float)inv_m;
            prm.coef->m = m;
            prm.result->j = 0;
            prm.result->status = sm.flag_timeout ? QN_ERR_DEVICE_TIMEOUT : QN_ERR_NONFINITE;
            prm.result->sweeps = 0;
            prm.result->redo = prm.only_if_redo ? 2 : 0;
            prm.result->tau_eff = prm.tau;
        }
        return;
    }

    // ---------------------------------------------------------------- phase 3: two-sided Jacobi
    // Round-robin ordering as a systolic array (Brent and Luk): the matrix is kept in the order of the tournament
    // table, pair k = physical positions (2k, 2k+1), so thread (a, b) always owns the 2x2 block at rows 2a, 2a+1 and
    // columns 2b, 2b+1, loads it with two 16-byte reads, and writes the rotated entries to where their rows and
    // columns move for the next round (position 0 stays, the other top positions 2k move right, the bottom
    // positions 2k+1 move left, the ends turn round).  M2-1 rounds per sweep bring every pair together once.  The
    // rounds read one copy of A and V and write the other.  (With the blocks addressed through the changing index
    // pairs instead, the scattered 8-byte accesses made the kernel shared-memory bound at about 1200 cycles per
    // round.)  The threads on the diagonal (a == b) compute their pair's rotation and publish (c, s): two
    // barriers per round.  The eigenvalues and the columns of V end up in tournament order, which phase 4 does
    // not care about; a padding index (odd m) never rotates and keeps its zero eigenvalue.
    const int M2 = m + (m & 1);
    const int H = M2 / 2;
    const int N = M2 - 1;
    const int jthreads = H * H > QN_MAX_M ? ((H * H + 31) / 32) * 32 : QN_MAX_M;  // threads that take part from here on
    if (M2 > m) {
        for (int e = tid; e < M2; e += nthr) {
            sm.A[m * kLd + e] = 0.0;
            sm.A[e * kLd + m] = 0.0;
        }
    }
    for (int e = tid; e < M2 * M2; e += nthr) sm.V[(e / M2) * kLd + (e % M2)] = (e / M2 == e % M2) ? 1.0 : 0.0;
    __syncthreads();
    double fro = 0.0;
    for (int e = tid; e < m * m; e += nthr) {
        const double a = sm.A[(e / m) * kLd + (e % m)];
        fro += a * a;
    }
    fro = sqrt(block_sum(fro, sm.red));

    // ---------------------------------------------------------------- phase 3a: fp32 pre-diagonalisation
    if (m >= kPreMinM && fro > 0.0) {
        const double scale = 1.0 / fro;
        for (int e = tid; e < M2 * M2; e += nthr) {
            const int k = e / M2, l = e % M2;
            sm.f.A[0][k * kLd + l] = (float)(sm.A[k * kLd + l] * scale);
            sm.f.V[0][k * kLd + l] = k == l ? 1.f : 0.f;
        }
        __syncthreads();
        int cur = 0;
        if (tid < jthreads) cur = jacobi_fp32(sm, M2, tid, jthreads);
        if (tid == 0) sm.j = cur;
        __syncthreads();
        cur = sm.j;
        __syncthreads();
        // Q = V32 (columns in tournament order) is orthogonal to about 1e-6 only; one Newton-Schulz step
        // Q <- Q (1.5 I - 0.5 Q^T Q) brings ||Q^T Q - I|| to about 1e-12.  A2 and V2 are free: scratch.
        for (int e = tid; e < M2 * M2; e += nthr) sm.V[(e / M2) * kLd + (e % M2)] = (double)sm.f.V[cur][(e / M2) * kLd + (e % M2)];
        __syncthreads();
        for (int e = tid; e < M2 * M2; e += nthr) {
            const int i = e / M2, l = e % M2;
            double acc = 0.0;
            for (int k = 0; k < M2; ++k) acc = fma(sm.V[k * kLd + i], sm.V[k * kLd + l], acc);
            sm.A2[i * kLd + l] = (i == l ? 1.5 : 0.0) - 0.5 * acc;
        }
        __syncthreads();
        for (int e = tid; e < M2 * M2; e += nthr) {
            const int i = e / M2, l = e % M2;
            double acc = 0.0;
            for (int k = 0; k < M2; ++k) acc = fma(sm.V[i * kLd + k], sm.A2[k * kLd + l], acc);
            sm.V2[i * kLd + l] = acc;
        }
        __syncthreads();
        for (int e = tid; e < M2 * M2; e += nthr) sm.V[(e / M2) * kLd + (e % M2)] = sm.V2[(e / M2) * kLd + (e % M2)];
        __syncthreads();
        // A <- Q^T A Q (symmetrised): nearly diagonal, in the order of Q's columns; the fp64 Jacobi continues from V = Q
        for (int e = tid; e < M2 * M2; e += nthr) {
            const int i = e / M2, l = e % M2;
            double acc = 0.0;
            for (int k = 0; k < M2; ++k) acc = fma(sm.A[i * kLd + k], sm.V[k * kLd + l], acc);
            sm.A2[i * kLd + l] = acc;
        }
        __syncthreads();
        for (int e = tid; e < M2 * M2; e += nthr) {
            const int i = e / M2, l = e % M2;
            double acc = 0.0;
            for (int k = 0; k < M2; ++k) acc = fma(sm.V[k * kLd + i], sm.A2[k * kLd + l], acc);
            sm.V2[i * kLd + l] = acc;
        }
        __syncthreads();
        for (int e = tid; e < M2 * M2; e += nthr) {
            const int i = e / M2, l = e % M2;
            sm.A[i * kLd + l] = 0.5 * (sm.V2[i * kLd + l] + sm.V2[l * kLd + i]);
        }
        __syncthreads();
    }
    // ---------------------------------------------------------------- phase 1b (learning-rate cap): Gram of theta
    if (prm.source == QN_SRC_PARTIALS) {
        const int E = tri_len + m;
        double* packed = sm.A2;  // free until the fp64 rounds start
        if (prm.tau_cap && prm.partials_theta) {
            // the same fixed-order sum for the Gram of theta; it stays reference-shifted: it is only ever applied
            // to retained v_k, which are orthogonal to the vector of ones, so the centring would change nothing
            for (int e = tid; e < tri_len; e += nthr) {
                double s0 = 0, s1 = 0;
                int p = 0;
                for (; p + 1 < prm.num_partials_theta; p += 2) {
                    s0 += prm.partials_theta[(int64_t)(p + 0) * E + e];
                    s1 += prm.partials_theta[(int64_t)(p + 1) * E + e];
                }
                if (p < prm.num_partials_theta) s0 += prm.partials_theta[(int64_t)p * E + e];
                packed[e] = s0 + s1;
            }
            __syncthreads();
            for (int e = tid; e < m * m; e += nthr) {
                const int k = e / m, l = e % m;
                sm.B[k * kLd + l] = packed[k <= l ? qn_tri_index(m, k, l) : qn_tri_index(m, l, k)];
            }
            __syncthreads();
        }
    }
    if (tid >= jthreads) return;  // the remaining phases synchronise with a named barrier over jthreads
    const double thresh = 1e-15 * fro;
    const double inv_fro = fro > 0.0 ? 1.0 / fro : 0.0;  // brings entries into fp32 range whatever the data's scale
    const int pa_idx = tid / H, pb_idx = tid % H;
    const bool worker = tid < H * H;
    const int ra = 2 * pa_idx, cb = 2 * pb_idx;  // this thread's block, every round
    const int nr0 = next_pos(ra, M2), nr1 = next_pos(ra + 1, M2), nc0 = next_pos(cb, M2), nc1 = next_pos(cb + 1, M2);
    double* Ar = sm.A;
    double* Aw = sm.A2;
    double* Vr = sm.V;
    double* Vw = sm.V2;
    int sweeps = 0;
    bool converged = (fro == 0.0) || m < 2;
    // Rotation that zeroes a_pq.  The angle comes from fp32 arithmetic on values scaled into fp32 range
    // (two MUFU reciprocal-square-roots and one reciprocal; relative error ~1e-7), so the rotation leaves
    // a'_pq = O(1e-7 a_pq), which the next sweep removes.  What must hold to fp64 accuracy is
    // c^2 + s^2 = 1: (c, s) are rescaled in fp64 by 1 - e/2 with e = c^2 + s^2 - 1 ~ 1e-7, which leaves
    // an error of 3e^2/8 ~ 4e-15 per rotation.  fp64 operations have a long dependent latency on this
    // part, so as few as possible sit on this chain.
    auto rotation = [&](double app, double aqq, double apq, double& c, double& s) {
        c = 1.0;
        s = 0.0;
        if (fabs(apq) > thresh) {
            const float df = (float)((aqq - app) * inv_fro);
            const float of = (float)((apq + apq) * inv_fro);
            const float r2 = fmaf(df, df, of * of);
            const float h = r2 * rsqrtf(r2);                                   // sqrt(d^2 + o^2)
            const float tf = copysignf(__fdividef(fabsf(of), fabsf(df) + h), df * of);  // tan(phi)
            const float cf = rsqrtf(fmaf(tf, tf, 1.0f));
            const double c0 = (double)cf, s0 = (double)(tf * cf);
            const double e = fma(c0, c0, fma(s0, s0, -1.0));
            const double k = fma(e, -0.5, 1.0);
            c = c0 * k;
            s = s0 * k;
        }
    };
    const int sweep_limit = prm.max_sweeps > 0 && prm.max_sweeps < kMaxSweeps ? prm.max_sweeps : kMaxSweeps;
    while (!converged && sweeps < sweep_limit) {
        for (int r = 0; r < N; ++r) {
            double x00 = 0.0, x01 = 0.0, x10 = 0.0, x11 = 0.0;
            if (worker) {
                const double2 r0 = *reinterpret_cast<const double2*>(&Ar[ra * kLd + cb]);
                const double2 r1 = *reinterpret_cast<const double2*>(&Ar[(ra + 1) * kLd + cb]);
                x00 = r0.x;
                x01 = r0.y;
                x10 = r1.x;
                x11 = r1.y;
                if (pa_idx == pb_idx) {  // the diagonal block holds a_pp, a_pq, a_qq of pair a
                    double c, s2;
                    rotation(x00, x11, x01, c, s2);
                    sm.rot_c[pa_idx] = c;
                    sm.rot_s[pa_idx] = s2;
                }
            }
            asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
            if (worker) {
                const double ca = sm.rot_c[pa_idx], sa = sm.rot_s[pa_idx];
                const double cbr = sm.rot_c[pb_idx], sbr = sm.rot_s[pb_idx];
                const double2 v0 = *reinterpret_cast<const double2*>(&Vr[ra * kLd + cb]);
                const double2 v1 = *reinterpret_cast<const double2*>(&Vr[(ra + 1) * kLd + cb]);
                // Y = J_a^T X J_b on this thread's 2x2 block
                const double t00 = cbr * x00 - sbr * x01, t01 = sbr * x00 + cbr * x01;
                const double t10 = cbr * x10 - sbr * x11, t11 = sbr * x10 + cbr * x11;
                double y00 = ca * t00 - sa * t10, y10 = sa * t00 + ca * t10;
                double y01 = ca * t01 - sa * t11, y11 = sa * t01 + ca * t11;
                if (pa_idx == pb_idx) y01 = y10 = 0.5 * (y01 + y10);  // keep the diagonal block symmetric
                Aw[nr0 * kLd + nc0] = y00;
                Aw[nr0 * kLd + nc1] = y01;
                Aw[nr1 * kLd + nc0] = y10;
                Aw[nr1 * kLd + nc1] = y11;
                // V <- V J_b on rows 2a, 2a+1 (the rows of V are not reordered, its columns move with A's)
                Vw[ra * kLd + nc0] = cbr * v0.x - sbr * v0.y;
                Vw[ra * kLd + nc1] = sbr * v0.x + cbr * v0.y;
                Vw[(ra + 1) * kLd + nc0] = cbr * v1.x - sbr * v1.y;
                Vw[(ra + 1) * kLd + nc1] = sbr * v1.x + cbr * v1.y;
            }
            asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
            double* t = Ar;
            Ar = Aw;
            Aw = t;
            t = Vr;
            Vr = Vw;
            Vw = t;
        }
        ++sweeps;
        // converged when no off-diagonal element exceeds the threshold (one pass over the matrix)
        int big = 0;
        for (int e = tid; e < M2 * M2; e += jthreads) {
            const int k = e / M2, l = e % M2;
            big |= (k != l) && (fabs(Ar[k * kLd + l]) > thresh);
        }
        big = __any_sync(0xffffffffu, big);
        if (big && (tid & 31) == 0) sm.flag_rotated = 1;
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
        const int rotated = sm.flag_rotated;
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");  // everyone has read the flag
        if (!rotated) converged = true;
        if (tid == 0) sm.flag_rotated = 0;
        // the barriers of the next sweep's first round order this reset before the next set
    }

    // ---------------------------------------------------------------- phase 4: sigma, j, d, c
    // all M2 positions take part: with odd m the padding index (eigenvalue exactly 0, never retained) may sit anywhere
    if (tid < M2) {
        const double mu = Ar[tid * kLd + tid];
        sm.mu[tid] = mu > QN_NOISE_FLOOR * sm.diag_scale ? mu : 0.0;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
    if (tid < M2) {
        const double mine = sm.mu[tid];
        int rank = 0;
        for (int l = 0; l < M2; ++l) {
            const double o = sm.mu[l];
            rank += (o > mine) || (o == mine && l < tid);
        }
        sm.order[rank] = tid;
        sm.sigma[rank] = sqrt(mine > 0.0 ? mine : 0.0);
    }
    asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
    if (tid == 0) {
        int j = 0;
        const double s1 = sm.sigma[0];
        if (s1 > 0.0)
            for (int k = 0; k < m; ++k) j += (sm.sigma[k] >= prm.lambda * s1 && sm.sigma[k] > 0.0);
        if (j > m - 1) j = m - 1;
        if (prm.j_cap >= 0 && j > prm.j_cap) j = prm.j_cap;  // the caller's cap on the number of modes
        sm.j = j;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
    const int j = sm.j;
    // Learning-rate cap (Section 3, last paragraph: tau_opt = 1 / sigma_max of the Hessian).  The operator is built
    // from Hbar y_k = sigma_k u_k, so the Hessian's largest singular value as the method sees it is
    // max_k sigma_k / ||y_k||, with ||y_k||^2 = v_k^T (Theta^T Theta) v_k.
    double tau_use = prm.tau;
    if (prm.tau_cap && prm.partials_theta && prm.source == QN_SRC_PARTIALS && j > 0 && prm.tau > 0.0) {
        for (int e = tid; e < j * m; e += jthreads) {  // the copy of A that is not current is free: scratch for the j x m products
            const int k = e / m, a = e % m, col = sm.order[k];
            double bv = 0.0;
            for (int b = 0; b < m; ++b) bv += sm.B[a * kLd + b] * Vr[b * kLd + col];
            Aw[k * kLd + a] = Vr[a * kLd + col] * bv;
        }
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
        if (tid < j) {
            double y2 = 0.0;
            for (int a = 0; a < m; ++a) y2 += Aw[tid * kLd + a];
            sm.d[tid] = y2 > 0.0 ? sm.sigma[tid] / sqrt(y2) : 0.0;
        }
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
        if (tid == 0) {
            double smax = 0.0;
            for (int k = 0; k < j; ++k) smax = fmax(smax, sm.d[k]);
            sm.tau_eff = (smax > 0.0 && 1.0 / smax < prm.tau) ? 1.0 / smax : prm.tau;
        }
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
        tau_use = sm.tau_eff;
        asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");  // d is rewritten below
    }
    if (tid < j) {
        const int col = sm.order[tid];
        double dot = 0.0;
        for (int k = 0; k < m; ++k) dot += Vr[k * kLd + col] * sm.w[k];
        sm.modec[tid] = dot / sm.mu[col];
    }
    asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
    if (tid < m) {
        double dk = 0.0;
        for (int r = 0; r < j; ++r) dk += Vr[tid * kLd + sm.order[r]] * sm.modec[r];
        sm.d[tid] = dk;
    }
    asm volatile("bar.sync 1, %0;" ::"r"(jthreads) : "memory");
    if (tid < QN_MAX_M) {
        double s = 0.0;
        for (int k = 0; k < m; ++k) s += sm.d[k];
        prm.coef->c[tid] = tid < m ? (float)(tau_use * (sm.d[tid] - s * inv_m)) : 0.f;
        prm.result->sigma[tid] = tid < m ? sm.sigma[tid] : 0.0;
    }
    if (tid == 0) {
        prm.coef->tau = (float)tau_use;
        prm.coef->inv_m = (float)inv_m;
        prm.coef->m = m;
        prm.result->tau_eff = tau_use;
        prm.result->j = j;
        prm.result->status = sm.flag_timeout ? QN_ERR_DEVICE_TIMEOUT : converged ? QN_OK : QN_ERR_NOT_CONVERGED;
        prm.result->sweeps = sweeps;
        // A reduced-precision Gram pass leaves an error of about redo_coeff * (sigma_1 / sigma_k)^2 on sigma_k: if
        // that is too much for the smallest retained one, ask for the pass to be repeated in fp64 (the sigma computed
        // here are good enough to decide: the trigger sits a factor of four below what the library promises).
        int redo = prm.only_if_redo ? 2 : 0;
        if (prm.redo_coeff > 0.0 && j > 0 && sm.sigma[j - 1] > 0.0) {
            const double ratio = sm.sigma[0] / sm.sigma[j - 1];
            if (prm.redo_coeff * ratio * ratio > QN_REDO_TRIGGER) redo = 1;
        }
        prm.result->redo = redo;
    }
}

}  // namespace qn

cudaError_t qn_solve_init() {
    return cudaFuncSetAttribute(qn::solve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                (int)sizeof(qn::SolveSmem));
}

cudaError_t qn_launch_solve(const qn_solve_params& p, cudaStream_t st, int* launches) {
    const int M2 = p.m + (p.m & 1);
    const int H = M2 / 2;
    (void)H;
    const int threads = 1024;  // the partial sums and the centring use all of them; the Jacobi phase H*H
    qn::solve_kernel<<<1, threads, sizeof(qn::SolveSmem), st>>>(p);
    cudaError_t e = cudaGetLastError();
    if (e == cudaSuccess && launches) *launches += 1;
    return e;
}
