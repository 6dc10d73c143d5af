// Internal declarations shared by the .cu files of libqn (not part of the public ABI).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "qn.h"

// Packed layout of one Gram partial for m Workers: the upper triangle of the (reference-shifted)
// Gram by rows, entry (k,l), k <= l, at k*m - k*(k-1)/2 + (l-k), followed by t[m] (the products of
// each shifted row with the per-column reference).
__host__ __device__ inline int qn_tri_index(int m, int k, int l) { return k * m - (k * (k - 1)) / 2 + (l - k); }
__host__ __device__ inline int qn_partial_len(int m) { return m * (m + 1) / 2 + m; }

// Below this n the Gram pass forms every product and sum in fp64 (see qn_gram.cu): with fp32 products
// the error of an eigenvalue is about 6e-8 * mu_1 / sqrt(n), which only falls under the 1e-10 * mu_1
// needed for sigma to be good to 1e-5 * sigma_1 on near-null modes once n is a few million.
#define QN_PRECISE_BELOW (int64_t(1) << 22)
// The tensor-core Gram pass (m > 8) starts earlier: its error does not depend on n (the truncating accumulation is a
// bias), a step checks it against the spectrum on the device and repeats the pass in fp64 where needed, and it is
// faster than the fp64 pass from a few ten thousand columns on even though a CTA then only gets a handful of stages
// (measured, whole step, m = 32: 139 against 158 us at n = 2^17, 162 against 243 us at 2^19; below 2^17 the two are
// within 5 % and the eigen-solve is nearly all of the step).
#ifndef QN_TC_MIN_N
#define QN_TC_MIN_N (int64_t(1) << 17)
#endif

// Eigenvalues of the centred Gram below this fraction of the largest diagonal entry of the
// uncentred (reference-shifted or raw) Gram are rounding noise of the m x m centring and are set to 0.
#define QN_NOISE_FLOOR 1.4e-14

// Device block read back by the host after a step.
struct qn_result_block {
    int32_t j;
    int32_t status;  // qn_status seen on the device (OK, NOT_CONVERGED, NONFINITE)
    int32_t sweeps;
    int32_t redo;    // bit 0: the spectrum asks for the Gram pass to be repeated in fp64 (set by the first solve, cleared
                     // by the second); bit 1: the results come from such a repeated pass
    double sigma[QN_MAX_M];
    double tau_eff;  // the learning rate the step used (tau, or less under the learning-rate cap)
};

// Coefficients consumed by the combine kernel:
// theta_new = mean(theta) - tau*mean(g) + sum_k c[k]*((g_k - g_0) - (theta_k - theta_0)).
struct qn_coef_block {
    float c[QN_MAX_M];
    float tau;
    float inv_m;
    int32_t m;
    int32_t pad;
};

// What the solve kernel starts from.
enum qn_solve_source {
    QN_SRC_PARTIALS = 0,  // sum `num_partials` packed partials; if raw_gram != NULL also store the sum there
    QN_SRC_WINDOW = 1,    // start from the raw Gram kept in `raw_gram` (reference 0, t = 0)
    QN_SRC_SUMMED = 2     // start from m*m + m doubles in `raw_gram`: a centred Gram followed by w = G^T gbar
};

struct qn_solve_params {
    int32_t m;
    int32_t source;
    const double* partials;  // [num_partials][qn_partial_len(m)]
    int32_t num_partials;
    double* raw_gram;     // m*m doubles read (QN_SRC_WINDOW), m*m + m read (QN_SRC_SUMMED), or m*m written with the
                          // uncentred sum (QN_SRC_PARTIALS)
    double* gram_out;     // m*m + m doubles: centred C then w (may be NULL)
    int32_t gram_only;    // stop after writing gram_out
    double tau, lambda;
    int32_t j_cap;        // < 0: no cap; else at most this many of the modes kept by the lambda rule
    int32_t max_sweeps;   // limit on the fp64 Jacobi sweeps (0: the built-in limit); reaching it gives QN_ERR_NOT_CONVERGED
    int32_t tau_cap;      // != 0 with partials_theta: tau <- min(tau, 1 / max_k sigma_k / ||Theta v_k||)
    const double* partials_theta;  // Gram partials of theta (same layout as `partials`), or NULL
    int32_t num_partials_theta;
    const double* rhs_raw;  // NULL, or m doubles g_k^T z: the coefficients are then built for z instead of gbar
                            // (w = P rhs_raw) and with tau = -1, i.e. for out = z - G d + Theta d (Eq. (4))
    double redo_coeff;    // > 0: the Gram came from a reduced-precision pass whose relative error on a retained sigma_k is
                          // about redo_coeff * (sigma_1 / sigma_k)^2; if that exceeds QN_REDO_TRIGGER for the smallest
                          // retained one, result->redo bit 0 is set (the step then repeats the pass in fp64)
    int32_t only_if_redo; // != 0: return at once unless result->redo bit 0 is set (the second solve of such a step)
    qn_coef_block* coef;
    qn_result_block* result;
    int* error_word;      // device int set by a kernel that gave up on a bounded wait (may be NULL); read and cleared
};

// Launchers.  Each returns the launch error and adds the kernels it launched to *launches.
// error_word (device int, may be NULL) is set to 1 by a kernel that gave up on a bounded wait.
// lambda_hint: the cut-off of the step that will use the Gram, or 0 if unknown.  From QN_REF0_MIN_LAMBDA on, the
// bulk-copy kernel for bf16 storage and m <= 8 may take Worker 0 instead of the mean as its per-column reference
// (a third fewer instructions; the error of a retained sigma_k grows as 1 / lambda^2, see qn_gram.cu).
#define QN_REF0_MIN_LAMBDA 0.01
// Predicted relative error of the smallest retained sigma above which the Gram pass is repeated in fp64 (a quarter
// of the 1e-5 the library promises), and the measured error coefficients of the reduced-precision passes (relative
// error of sigma_k = coefficient * (sigma_1 / sigma_k)^2 on inputs whose largest modes sit on few Workers):
//   tensor cores: the fp32 accumulator truncates each product, a bias proportional to the chain length and
//                 independent of n: 2e-9 for fp32 storage (chains of 8 instructions), 2e-8 for bf16 (16)
//   fp32 products on the plain ALUs: unbiased, 2e-10 at n = 2^22 (tiled and register-fed kernels) or 6e-10 (bulk-copy
//                 kernel, which adds 64 columns per accumulator in fp32) and falling as 1 / sqrt(n); the bulk-copy
//                 kernel with Worker 0 as its reference 2e-9 at n = 2^22
#define QN_REDO_TRIGGER 2.5e-6
#define QN_REDO_COEFF_TC_F32 2e-9
#define QN_REDO_COEFF_TC_BF16 2e-8
#define QN_REDO_COEFF_ALU_AT_4M 2e-10
#define QN_REDO_COEFF_BULK_AT_4M 6e-10
#define QN_REDO_COEFF_REF0_AT_4M 2e-9
// path: QN_GRAM_PATH_* of qn.h (qn_set_gram_path).
cudaError_t qn_launch_gram(qn_dtype dtype, const void* g, int64_t n, int m, bool raw, double* partials,
                           int* num_partials, int max_partials, cudaStream_t st, int* launches,
                           int* error_word = nullptr, double lambda_hint = 0.0, int path = QN_GRAM_PATH_AUTO,
                           int* kernel_out = nullptr,  // kernel_out: which kernel was dispatched (QN_KERNEL_* of qn.h)
                           const int* run_if = nullptr);  // run_if: the pass forms every product in fp64 on the plain
                                                          // ALUs and returns at once unless bit 0 of *run_if is set
// Error coefficient (see QN_REDO_TRIGGER) of the pass that `kernel` (QN_KERNEL_*) stands for; 0 for an fp64 pass.
double qn_gram_error_coeff(int kernel, qn_dtype dtype, int64_t n, double lambda_hint);
// Loads every Gram kernel variant into the current context (allocates nothing the caller can see later: after it,
// the first launch of a variant no longer loads code).
cudaError_t qn_gram_preload();
cudaError_t qn_gram_tc_preload();
cudaError_t qn_launch_wait_probe(int* error_word, cudaStream_t st);
bool qn_gram_tc_applicable(qn_dtype dtype, const void* g, int64_t n, int m);
cudaError_t qn_launch_gram_tc(qn_dtype dtype, const void* g, int64_t n, int m, double* partials, int* num_partials,
                              int max_partials, int* error_word, cudaStream_t st);
cudaError_t qn_launch_solve(const qn_solve_params& p, cudaStream_t st, int* launches);
// base == NULL: theta_new of Eq. (2).  base = z (n elements): out = z + sum_k c[k] * ((g_k - g_0) - (theta_k - theta_0)).
cudaError_t qn_launch_combine(qn_dtype dtype, const void* theta, const void* g, int64_t n, int m,
                              const qn_coef_block* coef, void* theta_new, cudaStream_t st, int* launches,
                              const void* base = nullptr);
// Row refresh of the asynchronous window: the products of g_col with the m rows of window_g (row `slot` is taken
// to be g_col itself), patched into row and column `slot` of raw_gram.  Lands g_col in window_row_out; if it can
// also land theta_col in theta_row_out (bulk-copy kernel) it sets *theta_landed, otherwise the caller copies that
// column itself.  With dots_out != NULL the m products go there instead (slot = -1, window_row_out = theta_col =
// NULL: nothing is landed), which is G^T z up to the centring for an arbitrary vector z.
cudaError_t qn_launch_row(qn_dtype dtype, const void* window_g, const void* g_col, void* window_row_out,
                          const void* theta_col, void* theta_row_out, int64_t n, int m, int slot, double* partials,
                          int max_partials, double* raw_gram, double* dots_out, unsigned int* ticket, int* error_word,
                          bool* theta_landed, cudaStream_t st, int* launches);
cudaError_t qn_solve_init();

int qn_sm_count();
