/*
 * qn_oracle.c -- slow, plain fp64 CPU evaluation of the Parameter-Server quasi-Newton step of
 * Arnold & Wang, "Accelerating SGD for Distributed Deep-Learning Using Approximated Hessian
 * Matrix" (arXiv 1709.05069), Section 2 (Method), Eq. (2)-(4).
 *
 * THIS IS TEST INFRASTRUCTURE.  It is the checker the CUDA library is compared with and the CPU
 * baseline that the benchmark times.  It is not part of the product path: nothing in the CUDA
 * library or its Python binding includes, links, imports or calls this file, and this file uses
 * nothing of theirs.  It follows the paper's definitions literally (explicit means, explicit
 * centred columns, explicit u_k, y_k, alpha_k, z-perp) and deliberately does not use the collapsed
 * "theta*a + g*b" form, so that the collapse itself is under test.
 *
 * Storage: theta[m][n], g[m][n], row k = Worker k (the transpose of the paper's n x m matrices,
 * whose k-th column is Worker k).  Elements are fp32 or bf16 bit patterns; each is promoted
 * exactly to fp64 and every sum, product, square root and division below is fp64.
 *
 * Pins (tests/test_oracle_pins.py): SGD special case (j = 0), Newton recovery on a quadratic,
 * orthonormal u_k, agreement with a library SVD of G, the secant property H^-1(sigma_k u_k) = y_k,
 * identity on the complement, the m = 2 closed form, the null vector of the centred Gram, the
 * collapsed form, symmetries, and a brute-force n x n construction of Eq. (3).
 * Every exported function is covered by at least one of them; none is "parity unpinned".
 *
 * Readings of the paper taken here (the paper is silent or loose on these points):
 *   - the Hermitian transpose is a plain transpose (real data);
 *   - sigma_1 >= ... >= sigma_m >= 0 are the square roots of the eigenvalues of G^T G, with tiny
 *     negative eigenvalues from round-off clamped to 0 before the root;
 *   - j = number of k with sigma_k >= lambda*sigma_1 and sigma_k > 0, never more than m - 1
 *     (centring makes G*1 = 0, so sigma_m is round-off only); j = 0 when sigma_1 = 0;
 *     lambda > 1 is accepted and gives j = 0 (the SGD special case);
 *   - u_k = G v_k / ||G v_k||_2 uses the norm computed from the data, p_k = y_k / sigma_k uses
 *     sigma_k from the eigenvalue, as the paper writes them;
 *   - u_k is never formed for k > j.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define QNO_F32 0
#define QNO_BF16 1
#define QNO_MAX_M 64
#define QNO_CHUNK 4096 /* columns per summation chunk */

static inline double qno_load(const void* base, int dtype, int64_t idx) {
    if (dtype == QNO_F32) return (double)((const float*)base)[idx];
    uint32_t u = (uint32_t)((const uint16_t*)base)[idx] << 16;
    float f;
    memcpy(&f, &u, 4);
    return (double)f;
}

/* Round fp64 to the storage type, round-to-nearest-even, one rounding. */
static inline uint16_t qno_to_bf16(double x) {
    if (isnan(x)) return 0x7fc0;
    /* fp64 -> fp32 with round-to-odd would be needed for an exact single rounding; instead round
       directly on the fp64 bits: bf16 keeps 8 significant bits. */
    if (x == 0.0 || isinf(x)) {
        float f = (float)x;
        uint32_t u;
        memcpy(&u, &f, 4);
        return (uint16_t)(u >> 16);
    }
    int e;
    double fr = frexp(fabs(x), &e); /* |x| = fr * 2^e, fr in [0.5,1) */
    int emin = -125;                /* smallest normal exponent in frexp convention (2^-126) */
    int shift = (e < emin) ? 8 - (emin - e) : 8; /* significant bits kept (subnormals keep fewer) */
    double r;
    if (shift <= -1) {
        r = 0.0; /* below half of the smallest subnormal */
    } else {
        double scaled = ldexp(fr, shift); /* in [2^(shift-1), 2^shift) */
        r = ldexp(nearbyint(scaled), -shift); /* default rounding mode: ties to even */
    }
    double y = ldexp(r, e);
    if (x < 0) y = -y;
    float f = (float)y; /* exact: y has at most 8 significant bits, or overflows to inf */
    uint32_t u;
    memcpy(&u, &f, 4);
    return (uint16_t)(u >> 16);
}

void qno_round_storage(int64_t n, int dtype, const double* in, void* out) {
    for (int64_t i = 0; i < n; ++i) {
        if (dtype == QNO_F32)
            ((float*)out)[i] = (float)in[i];
        else
            ((uint16_t*)out)[i] = qno_to_bf16(in[i]);
    }
}

/* Neumaier-compensated add of x into (s, c). */
static inline void qno_cadd(double* s, double* c, double x) {
    double t = *s + x;
    if (fabs(*s) >= fabs(x))
        *c += (*s - t) + x;
    else
        *c += (x - t) + *s;
    *s = t;
}

static int qno_threads(int nthreads) {
#ifdef _OPENMP
    if (nthreads <= 0) nthreads = omp_get_max_threads();
    return nthreads < 1 ? 1 : nthreads;
#else
    (void)nthreads;
    return 1;
#endif
}

int qno_threads_used(int nthreads) { return qno_threads(nthreads); }

/* Means of column i over the m Workers ("means" display of Section 2). */
static inline void qno_means(int64_t n, int m, int dtype, const void* theta, const void* g, int64_t i,
                             double* gbar, double* tbar) {
    double sg = 0.0, st = 0.0;
    for (int k = 0; k < m; ++k) {
        sg += qno_load(g, dtype, (int64_t)k * n + i);
        if (theta) st += qno_load(theta, dtype, (int64_t)k * n + i);
    }
    *gbar = sg / m;
    if (tbar) *tbar = st / m;
}

/*
 * Pass 1: C = G^T G (m x m), G[:,k] = grad J(theta_k) - gbar (Section 2, definition of G and the
 * matrix G^H G whose eigenvectors are V_G).  Chunked plain sums, compensated across chunks.
 */
int qno_gram(int64_t n, int m, int dtype, const void* g, double* C, int nthreads) {
    if (n < 1 || m < 1 || m > QNO_MAX_M) return 1;
    const int nt = qno_threads(nthreads);
    const int64_t nchunks = (n + QNO_CHUNK - 1) / QNO_CHUNK;
    const int mm = m * m;
    double* tot = (double*)calloc((size_t)nt * 2 * mm, sizeof(double));
    if (!tot) return 2;
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        const int tid = omp_get_thread_num();
#else
        const int tid = 0;
#endif
        double* s = tot + (size_t)tid * 2 * mm;
        double* c = s + mm;
        double part[QNO_MAX_M * QNO_MAX_M];
        double x[QNO_MAX_M];
        const int64_t c0 = nchunks * tid / nt, c1 = nchunks * (tid + 1) / nt;
        for (int64_t ch = c0; ch < c1; ++ch) {
            const int64_t i0 = ch * QNO_CHUNK, i1 = (i0 + QNO_CHUNK < n) ? i0 + QNO_CHUNK : n;
            memset(part, 0, sizeof(double) * mm);
            for (int64_t i = i0; i < i1; ++i) {
                double gbar;
                qno_means(n, m, dtype, NULL, g, i, &gbar, NULL);
                for (int k = 0; k < m; ++k) x[k] = qno_load(g, dtype, (int64_t)k * n + i) - gbar;
                for (int k = 0; k < m; ++k)
                    for (int l = k; l < m; ++l) part[k * m + l] += x[k] * x[l];
            }
            for (int k = 0; k < m; ++k)
                for (int l = k; l < m; ++l) qno_cadd(&s[k * m + l], &c[k * m + l], part[k * m + l]);
        }
    }
    for (int k = 0; k < m; ++k)
        for (int l = k; l < m; ++l) {
            double s = 0.0, c = 0.0;
            for (int t = 0; t < nt; ++t) {
                qno_cadd(&s, &c, tot[(size_t)t * 2 * mm + k * m + l]);
                qno_cadd(&s, &c, tot[(size_t)t * 2 * mm + mm + k * m + l]);
            }
            C[k * m + l] = C[l * m + k] = s + c;
        }
    free(tot);
    return 0;
}

/*
 * Eigen-decomposition of the symmetric m x m matrix A by cyclic Jacobi rotations: on return
 * mu[0] >= mu[1] >= ... and column k of V (V[r*m + k], r = row) is the unit eigenvector of mu[k]
 * (the first m columns of V_G and the squares of the diagonal of Sigma_G, Section 2).
 * Stops when the off-diagonal Frobenius norm is <= 1e-15 * ||A||_F, or after 100 sweeps (then
 * returns 3).
 */
int qno_eig(int m, const double* A_in, double* V, double* mu) {
    if (m < 1 || m > QNO_MAX_M) return 1;
    double A[QNO_MAX_M * QNO_MAX_M];
    memcpy(A, A_in, sizeof(double) * m * m);
    for (int r = 0; r < m; ++r)
        for (int c = 0; c < m; ++c) V[r * m + c] = (r == c) ? 1.0 : 0.0;
    double fro = 0.0;
    for (int r = 0; r < m * m; ++r) fro += A[r] * A[r];
    fro = sqrt(fro);
    int rc = 3;
    for (int sweep = 0; sweep < 100; ++sweep) {
        double off = 0.0;
        for (int p = 0; p < m; ++p)
            for (int q = 0; q < m; ++q)
                if (p != q) off += A[p * m + q] * A[p * m + q];
        if (sqrt(off) <= 1e-15 * fro) {
            rc = 0;
            break;
        }
        for (int p = 0; p < m - 1; ++p)
            for (int q = p + 1; q < m; ++q) {
                const double apq = A[p * m + q];
                if (apq == 0.0) continue;
                const double app = A[p * m + p], aqq = A[q * m + q];
                /* rotation angle that zeroes A[p][q]: tan(2 phi) = 2 apq / (aqq - app) */
                const double zeta = (aqq - app) / (2.0 * apq);
                const double t = (zeta >= 0 ? 1.0 : -1.0) / (fabs(zeta) + sqrt(1.0 + zeta * zeta));
                const double cs = 1.0 / sqrt(1.0 + t * t), sn = t * cs;
                for (int r = 0; r < m; ++r) { /* A <- A J */
                    const double arp = A[r * m + p], arq = A[r * m + q];
                    A[r * m + p] = cs * arp - sn * arq;
                    A[r * m + q] = sn * arp + cs * arq;
                }
                for (int c = 0; c < m; ++c) { /* A <- J^T A */
                    const double apc = A[p * m + c], aqc = A[q * m + c];
                    A[p * m + c] = cs * apc - sn * aqc;
                    A[q * m + c] = sn * apc + cs * aqc;
                }
                for (int r = 0; r < m; ++r) { /* V <- V J */
                    const double vrp = V[r * m + p], vrq = V[r * m + q];
                    V[r * m + p] = cs * vrp - sn * vrq;
                    V[r * m + q] = sn * vrp + cs * vrq;
                }
            }
    }
    /* sort descending by eigenvalue (selection sort, columns of V follow) */
    for (int k = 0; k < m; ++k) mu[k] = A[k * m + k];
    for (int k = 0; k < m - 1; ++k) {
        int best = k;
        for (int l = k + 1; l < m; ++l)
            if (mu[l] > mu[best]) best = l;
        if (best != k) {
            double tmp = mu[k];
            mu[k] = mu[best];
            mu[best] = tmp;
            for (int r = 0; r < m; ++r) {
                tmp = V[r * m + k];
                V[r * m + k] = V[r * m + best];
                V[r * m + best] = tmp;
            }
        }
    }
    return rc;
}

/* sigma_k = sqrt(max(mu_k, 0)); j per the lambda rule of Section 2 (text after Eq. (3)). */
int qno_cutoff(int m, const double* mu, double lambda, double* sigma) {
    for (int k = 0; k < m; ++k) sigma[k] = sqrt(mu[k] > 0.0 ? mu[k] : 0.0);
    int j = 0;
    if (sigma[0] > 0.0)
        for (int k = 0; k < m; ++k)
            if (sigma[k] >= lambda * sigma[0] && sigma[k] > 0.0) ++j;
    if (j > m - 1) j = m - 1;
    return j;
}

/*
 * Pass 2: for k = 1..j the norms ||G v_k||_2 and the projections alpha_k = z^T u_k with
 * u_k = G v_k / ||G v_k||_2 (Section 2, definition of u_k and the z-decomposition display).
 * z = NULL means z = gbar (the vector Eq. (2) applies the operator to).
 */
static int qno_project(int64_t n, int m, int dtype, const void* g, const double* V, int j, const double* z,
                       double* gvnorm, double* alpha, int nthreads) {
    if (j == 0) return 0;
    const int nt = qno_threads(nthreads);
    const int64_t nchunks = (n + QNO_CHUNK - 1) / QNO_CHUNK;
    double* tot = (double*)calloc((size_t)nt * 4 * QNO_MAX_M, sizeof(double));
    if (!tot) return 2;
#pragma omp parallel num_threads(nt)
    {
#ifdef _OPENMP
        const int tid = omp_get_thread_num();
#else
        const int tid = 0;
#endif
        double* sn = tot + (size_t)tid * 4 * QNO_MAX_M; /* sum, comp of ||Gv||^2 */
        double* cn = sn + QNO_MAX_M;
        double* sd = cn + QNO_MAX_M; /* sum, comp of z.(Gv) */
        double* cd = sd + QNO_MAX_M;
        double x[QNO_MAX_M], pn[QNO_MAX_M], pd[QNO_MAX_M];
        const int64_t c0 = nchunks * tid / nt, c1 = nchunks * (tid + 1) / nt;
        for (int64_t ch = c0; ch < c1; ++ch) {
            const int64_t i0 = ch * QNO_CHUNK, i1 = (i0 + QNO_CHUNK < n) ? i0 + QNO_CHUNK : n;
            for (int k = 0; k < j; ++k) pn[k] = pd[k] = 0.0;
            for (int64_t i = i0; i < i1; ++i) {
                double gbar;
                qno_means(n, m, dtype, NULL, g, i, &gbar, NULL);
                for (int l = 0; l < m; ++l) x[l] = qno_load(g, dtype, (int64_t)l * n + i) - gbar;
                const double zi = z ? z[i] : gbar;
                for (int k = 0; k < j; ++k) {
                    double gv = 0.0;
                    for (int l = 0; l < m; ++l) gv += x[l] * V[l * m + k];
                    pn[k] += gv * gv;
                    pd[k] += zi * gv;
                }
            }
            for (int k = 0; k < j; ++k) {
                qno_cadd(&sn[k], &cn[k], pn[k]);
                qno_cadd(&sd[k], &cd[k], pd[k]);
            }
        }
    }
    for (int k = 0; k < j; ++k) {
        double s1 = 0, c1 = 0, s2 = 0, c2 = 0;
        for (int t = 0; t < nt; ++t) {
            const double* b = tot + (size_t)t * 4 * QNO_MAX_M;
            qno_cadd(&s1, &c1, b[k]);
            qno_cadd(&s1, &c1, b[QNO_MAX_M + k]);
            qno_cadd(&s2, &c2, b[2 * QNO_MAX_M + k]);
            qno_cadd(&s2, &c2, b[3 * QNO_MAX_M + k]);
        }
        gvnorm[k] = sqrt(s1 + c1);
        alpha[k] = (s2 + c2) / gvnorm[k];
    }
    free(tot);
    return 0;
}

/*
 * Pass 3, one column i: Eq. (4), Hinv z = z_perp + sum_{k<=j} alpha_k sigma_k^-1 y_k with
 * z_perp = z - sum alpha_k u_k, y_k = Theta v_k.  Returns (Hinv z)_i; also gives thetabar_i.
 */
static inline double qno_hinv_column(int64_t n, int m, int dtype, const void* theta, const void* g,
                                     const double* V, int j, const double* sigma, const double* gvnorm,
                                     const double* alpha, const double* z, int64_t i, double* tbar_out) {
    double gbar, tbar;
    double x[QNO_MAX_M], th[QNO_MAX_M];
    qno_means(n, m, dtype, theta, g, i, &gbar, &tbar);
    for (int l = 0; l < m; ++l) {
        x[l] = qno_load(g, dtype, (int64_t)l * n + i) - gbar;      /* G[i][l] */
        th[l] = qno_load(theta, dtype, (int64_t)l * n + i) - tbar; /* Theta[i][l] */
    }
    const double zi = z ? z[i] : gbar;
    double zperp = zi, corr = 0.0;
    for (int k = 0; k < j; ++k) {
        double gv = 0.0, y = 0.0;
        for (int l = 0; l < m; ++l) {
            gv += x[l] * V[l * m + k];
            y += th[l] * V[l * m + k];
        }
        const double u = gv / gvnorm[k];
        zperp -= alpha[k] * u;
        corr += alpha[k] * (y / sigma[k]);
    }
    if (tbar_out) *tbar_out = tbar;
    return zperp + corr;
}

/* Shared front end: Gram, eigenpairs, cut-off, projections. */
static int qno_front(int64_t n, int m, int dtype, const void* g, double lambda, int j_cap, const double* z, double* V,
                     double* sigma, int* j_out, double* gvnorm, double* alpha, int nthreads) {
    double C[QNO_MAX_M * QNO_MAX_M], mu[QNO_MAX_M];
    int rc = qno_gram(n, m, dtype, g, C, nthreads);
    if (rc) return rc;
    rc = qno_eig(m, C, V, mu);
    if (rc) return rc;
    int j = qno_cutoff(m, mu, lambda, sigma);
    /* optional cap on the number of modes kept (the parameter j of Section 2 set from outside; Section 3
       stresses how much the result depends on it): the j_cap largest of those the lambda rule keeps */
    if (j_cap >= 0 && j > j_cap) j = j_cap;
    *j_out = j;
    return qno_project(n, m, dtype, g, V, j, z, gvnorm, alpha, nthreads);
}

/*
 * The Server step, Eq. (2): theta_new = thetabar - tau * Hinv gbar.
 *   theta, g      [m][n] storage-dtype bits (row k = Worker k)
 *   theta_new     n doubles (may be NULL)
 *   sample_idx    if non-NULL, only these ns columns are evaluated in pass 3 and theta_new has
 *                 ns entries (for full-size inputs where only sampled outputs are compared)
 *   sigma[m], V[m*m] (row-major, column k = v_k), alpha[m] (first j valid): optional outputs
 * Returns 0, or 1 bad argument, 2 out of memory, 3 Jacobi did not converge.
 */
/*
 * tau_cap != 0: the learning rate is bounded by the reciprocal of the largest singular value of the Hessian as
 * the method itself sees it (last paragraph of Section 3: tau_opt = 1 / sigma_max, "we directly approximate
 * sigma_max").  The operator is built from the pairs Hbar y_k = sigma_k u_k (Eq. (1) and the text before
 * Eq. (3)), so the estimate is max_{k<=j} ||Hbar y_k|| / ||y_k|| = max_k sigma_k / ||Theta v_k||_2, and
 * tau_eff = min(tau, 1 / that) for tau > 0.  tau_eff_out (may be NULL) receives the rate that was used.
 */
int qno_update_capped(int64_t n, int m, int dtype, const void* theta, const void* g, double tau, double lambda,
                      int j_cap, int tau_cap, double* theta_new, const int64_t* sample_idx, int64_t ns, int* j_out,
                      double* sigma_out, double* V_out, double* alpha_out, double* tau_eff_out, int nthreads) {
    if (n < 1 || m < 1 || m > QNO_MAX_M || !(lambda > 0.0)) return 1;
    double V[QNO_MAX_M * QNO_MAX_M], sigma[QNO_MAX_M], gvnorm[QNO_MAX_M], alpha[QNO_MAX_M];
    int j = 0;
    int rc = qno_front(n, m, dtype, g, lambda, j_cap, NULL, V, sigma, &j, gvnorm, alpha, nthreads);
    if (rc) return rc;
    if (tau_cap && j > 0 && tau > 0.0) {
        double ynorm[QNO_MAX_M], unused[QNO_MAX_M];
        rc = qno_project(n, m, dtype, theta, V, j, NULL, ynorm, unused, nthreads); /* ||Theta v_k||_2 */
        if (rc) return rc;
        double smax = 0.0;
        for (int k = 0; k < j; ++k)
            if (ynorm[k] > 0.0 && sigma[k] / ynorm[k] > smax) smax = sigma[k] / ynorm[k];
        if (smax > 0.0 && 1.0 / smax < tau) tau = 1.0 / smax;
    }
    if (tau_eff_out) *tau_eff_out = tau;
    if (theta_new) {
        const int64_t cnt = sample_idx ? ns : n;
        const int nt = qno_threads(nthreads);
#pragma omp parallel for num_threads(nt) schedule(static)
        for (int64_t s = 0; s < cnt; ++s) {
            const int64_t i = sample_idx ? sample_idx[s] : s;
            double tbar;
            const double h = qno_hinv_column(n, m, dtype, theta, g, V, j, sigma, gvnorm, alpha, NULL, i, &tbar);
            theta_new[s] = tbar - tau * h;
        }
    }
    if (j_out) *j_out = j;
    if (sigma_out) memcpy(sigma_out, sigma, sizeof(double) * m);
    if (V_out) memcpy(V_out, V, sizeof(double) * m * m);
    if (alpha_out) {
        memset(alpha_out, 0, sizeof(double) * m);
        memcpy(alpha_out, alpha, sizeof(double) * j);
    }
    return 0;
}

/* The Server step with the lambda rule alone (no cap on j). */
int qno_update(int64_t n, int m, int dtype, const void* theta, const void* g, double tau, double lambda,
               double* theta_new, const int64_t* sample_idx, int64_t ns, int* j_out, double* sigma_out,
               double* V_out, double* alpha_out, int nthreads) {
    return qno_update_capped(n, m, dtype, theta, g, tau, lambda, -1, 0, theta_new, sample_idx, ns, j_out, sigma_out,
                             V_out, alpha_out, NULL, nthreads);
}

/* Eq. (3)/(4) applied to an arbitrary z in R^n (n doubles): out = Hinv z. */
int qno_apply_hinv(int64_t n, int m, int dtype, const void* theta, const void* g, double lambda,
                   const double* z, double* out, int* j_out, int nthreads) {
    if (n < 1 || m < 1 || m > QNO_MAX_M || !(lambda > 0.0) || !z || !out) return 1;
    double V[QNO_MAX_M * QNO_MAX_M], sigma[QNO_MAX_M], gvnorm[QNO_MAX_M], alpha[QNO_MAX_M];
    int j = 0;
    int rc = qno_front(n, m, dtype, g, lambda, -1, z, V, sigma, &j, gvnorm, alpha, nthreads);
    if (rc) return rc;
    for (int64_t i = 0; i < n; ++i)
        out[i] = qno_hinv_column(n, m, dtype, theta, g, V, j, sigma, gvnorm, alpha, z, i, NULL);
    if (j_out) *j_out = j;
    return 0;
}

/*
 * The first j left vectors and images, written out in full for small n:
 * U[i*j + k] = (u_k)_i, Y[i*j + k] = (y_k)_i = (Theta v_k)_i  (Section 2, u_k and y_k).
 */
int qno_left_vectors(int64_t n, int m, int dtype, const void* theta, const void* g, double lambda, double* U,
                     double* Y, double* sigma_out, int* j_out) {
    if (n < 1 || m < 1 || m > QNO_MAX_M || !(lambda > 0.0)) return 1;
    double V[QNO_MAX_M * QNO_MAX_M], sigma[QNO_MAX_M], gvnorm[QNO_MAX_M], alpha[QNO_MAX_M];
    int j = 0;
    int rc = qno_front(n, m, dtype, g, lambda, -1, NULL, V, sigma, &j, gvnorm, alpha, 1);
    if (rc) return rc;
    for (int64_t i = 0; i < n; ++i) {
        double gbar, tbar;
        qno_means(n, m, dtype, theta, g, i, &gbar, &tbar);
        for (int k = 0; k < j; ++k) {
            double gv = 0.0, y = 0.0;
            for (int l = 0; l < m; ++l) {
                gv += (qno_load(g, dtype, (int64_t)l * n + i) - gbar) * V[l * m + k];
                y += (qno_load(theta, dtype, (int64_t)l * n + i) - tbar) * V[l * m + k];
            }
            U[i * j + k] = gv / gvnorm[k];
            Y[i * j + k] = y;
        }
    }
    if (sigma_out) memcpy(sigma_out, sigma, sizeof(double) * m);
    if (j_out) *j_out = j;
    return 0;
}
