/*
 * qn.h -- C ABI of the B200 (sm_100a) Parameter-Server quasi-Newton step of Arnold & Wang,
 * "Accelerating SGD for Distributed Deep-Learning Using Approximated Hessian Matrix"
 * (arXiv 1709.05069), Section 2 (Method).
 *
 * What one call computes (Section 2, Eq. (2)-(4)).  Given m Workers' parameter vectors
 * theta_k in R^n and gradients g_k = grad J(theta_k):
 *     gbar, thetabar      means over the Workers                         (display before Eq. (2))
 *     G, Theta            n x m, columns g_k - gbar and theta_k - thetabar
 *     G^T G = V diag(sigma^2) V^T,  sigma_1 >= ... >= sigma_m >= 0       (SVD paragraph)
 *     j                   sigma_j >= lambda sigma_1 > sigma_{j+1}        (text after Eq. (3))
 *     u_k = G v_k / ||G v_k||,  y_k = Theta v_k,  alpha_k = gbar^T u_k   (k = 1..j)
 *     theta_new = thetabar - tau ( gbar - sum alpha_k u_k + sum alpha_k sigma_k^-1 y_k )   Eq. (2),(4)
 * and j = 0 gives plain SGD, thetabar - tau gbar (sentence after Eq. (4)).
 *
 * Layout.  All matrices are Worker-major: theta[m][n] and g[m][n], row k = Worker k, each row
 * contiguous (the transpose of the paper's n x m matrices).  Elements are fp32 or bf16
 * (qn_dtype).  Arithmetic: the Gram pass forms fp64 products below 2^22 parameters and fp32 products
 * (m <= 8) or tensor-core products of a bf16 hi/lo split (m > 8, from 2^17 parameters on) above, always
 * with fp64 accumulation across work items, and is repeated in fp64 when the spectrum needs it (see
 * qn_update); the m x m eigen-problem and the coefficients are fp64; the final combination is fp32 with
 * one round-to-nearest-even to the storage type when theta_new is written.
 *
 * Pointers.  Unless a parameter says HOST, data pointers are DEVICE pointers on the device that
 * was current when the handle was created.  The caller owns every buffer it passes; the library
 * only reads inputs and only writes the named outputs.  The handle owns its workspace.
 * Rows that start on 16-byte boundaries (base pointer 16-byte aligned and n * element size a
 * multiple of 16) take the vectorised path; anything else takes a slower element-wise path,
 * never an error.  For full speed let every row start on a 128-byte boundary (n a multiple of 32
 * for fp32 storage, of 64 for bf16): rows that only meet the 16-byte rule were measured 8 to 15 %
 * slower, because every request of a streaming pass then touches one more cache line.
 *
 * Streams.  `cuda_stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 * Calls enqueue work on that stream and return without waiting unless they have to hand a HOST
 * result back (j_out / sigma_out non-NULL, qn_status_sync, qn_update_host).  All calls on one handle
 * share its workspace (partial sums, coefficients, result block): they must be ordered on the device,
 * i.e. issued on one stream or on streams that the caller orders with events.  Two steps of one handle
 * that overlap on the GPU race; use one handle per concurrent stream.
 *
 * Devices.  Every DEVICE pointer must point into memory of the handle's device (or managed memory);
 * a host pointer or another GPU's memory is refused with QN_ERR_INVALID before anything is launched.
 *
 * Errors.  Every call returns a qn_status; nothing throws or aborts.  Arguments are validated on
 * the host before anything is launched.  Conditions only the device can see (a non-finite Gram,
 * the Jacobi sweep limit, a bounded device wait that ran out) are recorded in a device status word that is returned by the next call
 * that synchronises; in both cases theta_new is still written (with j = 0, i.e. the SGD update,
 * for a non-finite Gram).
 *
 * There is no CPU fallback: without a usable CUDA device qn_create fails with QN_ERR_CUDA.
 */
#ifndef QN_H
#define QN_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define QN_MAX_M 64 /* largest supported number of Workers */

#if defined(__GNUC__)
#define QN_API __attribute__((visibility("default")))
#else
#define QN_API
#endif

typedef struct qn_ctx* qn_handle;

typedef enum { QN_F32 = 0, QN_BF16 = 1 } qn_dtype;

typedef enum {
    QN_OK = 0,
    QN_ERR_INVALID = 1,       /* bad argument (null, n < 1, m outside [1, QN_MAX_M], lambda <= 0, ...) */
    QN_ERR_ALLOC = 2,         /* device or host allocation failed */
    QN_ERR_CUDA = 3,          /* a CUDA runtime call failed (no device, launch error, ...) */
    QN_ERR_STATE = 4,         /* call not valid in the handle's state (window not full, ...) */
    QN_ERR_NOT_CONVERGED = 5, /* Jacobi hit its sweep limit; results were still written */
    QN_ERR_NONFINITE = 6,     /* Gram contained NaN/Inf; theta_new written with j = 0 */
    QN_ERR_DEVICE_TIMEOUT = 7 /* a kernel's bounded wait ran out; theta_new written with j = 0 */
} qn_status;

/* Human-readable text for a status code (static storage, never NULL). */
QN_API const char* qn_strerror(qn_status s);

/*
 * Create a handle for n parameters, m Workers and the given storage type on the CURRENT CUDA
 * device, and allocate its workspace there (a few MB; the asynchronous window is allocated by
 * the first qn_push).  1 <= m <= QN_MAX_M, n >= 1.  *out is set only on QN_OK.
 */
QN_API qn_status qn_create(int64_t n, int32_t m, qn_dtype dtype, qn_handle* out);

/* Free the handle and everything it owns.  Waits for the device to finish work it enqueued. */
QN_API qn_status qn_destroy(qn_handle h);

/*
 * Synchronous mode: the whole Server step (Section 2, Eq. (2)-(4)) on all m Workers at once.
 *   theta, g     [m][n], read-only
 *   tau          learning rate of Eq. (2), finite
 *   lambda       cut-off of the text after Eq. (3); > 0 and finite.  0 < lambda < 1 is the paper's
 *                range; lambda > 1 is accepted and keeps no mode (j = 0, the SGD update)
 *   theta_new    [n], written; must not overlap the inputs
 *   j_out        HOST int32, may be NULL
 *   sigma_out    HOST double[m], descending, may be NULL
 * If both j_out and sigma_out are NULL the call does not wait for the device.
 * Accuracy against the exact fp64 evaluation of Eq. (2)-(4) on the stored values: j exact when no sigma_k
 * lies within 1e-5 sigma_1 of lambda sigma_1; every sigma_k within 1e-5 sigma_1, the retained ones within a
 * relative 1e-5; theta_new within a relative L2 error of 1e-5 (fp32 storage) or 2e-3 (bf16 storage: the single
 * rounding of the output).  The first Gram pass is chosen from n, m, the storage type and lambda (fp64 products
 * below 2^22 parameters, or 2^17 with m > 8; fp32 or tensor-core products above), never from the data.
 * How the sigma figures are kept where the Gram pass rounds: fp32 products on the plain ALUs
 * (unbiased; the relative error of a retained sigma_k is about 2e-10 (sigma_1 / sigma_k)^2 at n = 2^22 and falls as
 * 1 / sqrt(n)), or for m > 8 the tensor cores, whose fp32 accumulator truncates each product: measured, a retained
 * sigma_k comes out low by about 2e-9 (fp32 storage) or 2e-8 (bf16 storage) times (sigma_1 / sigma_k)^2, whatever n.
 * Whether that is within the promise depends on the spectrum, so it is checked on the device: the eigen-solve compares
 * the smallest retained sigma_k with the pass's error coefficient (a factor of four inside 1e-5), and where it falls
 * short the Gram pass is repeated with every product in fp64 and the solve re-run, before the pass that writes
 * theta_new; nothing waits on the host.  A step therefore launches three kernels, or five of which two return at once
 * (when lambda is so small that some spectrum could need the repeat), and costs two to ten times more on inputs that do
 * need it.  qn_update, qn_update_host and qn_apply_hinv work this way; qn_gram and qn_update_from_gram do not see the
 * spectrum before the caller's reduction (see QN_GRAM_PATH_FP64), and the asynchronous window forms fp32 products.
 */
QN_API qn_status qn_update(qn_handle h, const void* theta, const void* g, double tau, double lambda,
                    void* theta_new, int32_t* j_out, double* sigma_out, void* cuda_stream);

/*
 * Cap on the number of modes: later steps on this handle keep at most j_cap of the modes that the lambda rule
 * retains (the largest singular values); j_cap < 0 removes the cap (the default), j_cap = 0 gives the plain
 * averaged-gradient step theta_bar - tau * g_bar (sentence after Eq. (4)).  Section 2 defines j through lambda
 * only; Section 3 reports that the result depends strongly on how many singular values are considered, so the
 * number can also be bounded directly.  sigma is still reported in full.  Host-side setting, no device work.
 */
QN_API qn_status qn_set_rank_cap(qn_handle h, int32_t j_cap);

/*
 * Limit on the fp64 Jacobi sweeps of the eigen-solve (Section 2 leaves the eigen-solver open; this library uses
 * cyclic Jacobi with a built-in limit of 30 sweeps, far above the 2 to 10 it needs).  max_sweeps = 0 restores the
 * built-in limit.  A step that reaches the limit before every off-diagonal entry is below 1e-15 of the matrix
 * norm still writes theta_new, j and sigma from the matrix as it stands and reports QN_ERR_NOT_CONVERGED.  Use:
 * a bound on the step's latency, and a way to see that status in a test.  Host-side setting, no device work.
 */
QN_API qn_status qn_set_sweep_limit(qn_handle h, int32_t max_sweeps);

/*
 * Which kernels the Gram pass may use (the paper has no counterpart; for A/B measurements and tests).
 *   QN_GRAM_PATH_AUTO       the default: tensor-core kernel for m > 8, bulk-copy kernel for m <= 8, both from
 *                           2^22 parameters on aligned rows; the register-fed plain-ALU kernels elsewhere
 *   QN_GRAM_PATH_PLAIN_ALU  the register-fed plain-ALU kernels everywhere (same results within the stated accuracy)
 *   QN_GRAM_PATH_FP64       the plain-ALU kernels with every product and sum in fp64 whatever n (several times slower
 *                           than the others above 2^22 parameters): for qn_gram / qn_update_from_gram callers whose
 *                           spectrum has retained modes far below sigma_1 (see the accuracy notes of those calls)
 * Host-side setting of the handle; nothing is read from the environment.
 */
#define QN_GRAM_PATH_AUTO 0
#define QN_GRAM_PATH_PLAIN_ALU 1
#define QN_GRAM_PATH_FP64 2
QN_API qn_status qn_set_gram_path(qn_handle h, int32_t path);

/*
 * Learning-rate cap (Section 3, last paragraph: the optimal rate is 1 / sigma_max of the Hessian, and the method
 * approximates sigma_max itself, so the rate can be bounded by it at every update).  The operator is built from
 * the pairs Hbar y_k = sigma_k u_k with y_k = Theta v_k (Eq. (1), text before Eq. (3)); the Hessian's largest
 * singular value as the method sees it is max_{k<=j} sigma_k / ||y_k||_2, and with the cap on, qn_update and
 * qn_update_host use tau_eff = min(tau, 1 / that) when tau > 0.  ||y_k||^2 = v_k^T (Theta^T Theta) v_k needs the
 * Gram of theta: one more streaming pass (m*n elements read, a fourth kernel launch).  The asynchronous window,
 * qn_update_from_gram and qn_apply_hinv ignore the setting.
 *   on           0 = off (default), else on; the first switch-on allocates the pass's partial sums on the device
 * qn_last_tau returns the rate used by the most recent step whose results were fetched to the host
 * (j_out or sigma_out non-NULL, or qn_status_sync).
 */
QN_API qn_status qn_set_tau_cap(qn_handle h, int32_t on);
QN_API double qn_last_tau(qn_handle h);

/*
 * The operator itself on an arbitrary vector: out = Hbar^{-1} z by Eq. (3)/(4),
 *   Hbar^{-1} z = z - sum_{k<=j} (u_k^T z) u_k + sum_{k<=j} (u_k^T z) sigma_k^{-1} y_k,
 * with u_k, y_k, sigma_k and the cut-off j built from (theta, g) exactly as in qn_update (qn_update is this
 * operator applied to z = gbar inside Eq. (2)).  Use: preconditioning a momentum or an averaged gradient, or
 * checking the secant property Hbar^{-1}(sigma_k u_k) = y_k.  Like the update, the two sums collapse onto one
 * m-vector d = sum_{k<=j} v_k (v_k^T G^T z) / sigma_k^2 and out = z - G d + Theta d.  Four kernels: g_k^T z for
 * all k (reads m*n + n elements), the Gram pass, the eigen-solve, one streaming pass that writes out.
 *   theta, g     as for qn_update
 *   z            DEVICE, n elements of the handle's dtype, read only
 *   out          DEVICE, n elements, must not overlap theta, g or z
 *   j_out, sigma_out   as for qn_update
 * Errors as for qn_update (lambda must be finite and > 0).
 */
QN_API qn_status qn_apply_hinv(qn_handle h, const void* theta, const void* g, double lambda, const void* z, void* out,
                               int32_t* j_out, double* sigma_out, void* cuda_stream);

/*
 * The reductions alone: the centred Gram C = G^T G (m x m, row-major, symmetric) followed by
 * w = G^T gbar (m values), as m*m + m doubles written to the DEVICE buffer gram_out
 * (Section 2: the matrix G^H G of the SVD paragraph, and the numerators of alpha_k = z^H u_k
 * for z = gbar).  The means and the centred columns are formed on the fly and never stored.
 */
QN_API qn_status qn_gram(qn_handle h, const void* g, double* gram_out, void* cuda_stream);

/*
 * The step with the Gram supplied by the caller: eigen-solve, cut-off and coefficients from `gram`, then the
 * streaming pass that writes theta_new (Eq. (2) with Eq. (4); everything of qn_update but its first pass).
 *
 * This is the n-sharded form of the Server step for several GPUs.  Each rank holds a slice of the columns of
 * all m Workers (theta, g: [m][n_local]) and a handle created for n_local.  Every sum over the parameter
 * index in Section 2 (G^H G and z^H u_k for z = gbar) is a sum over the slices, and the centring is linear, so:
 *   1. every rank calls qn_gram on its slice: m*m + m doubles (centred Gram of the slice, then G^T gbar);
 *   2. the caller adds these buffers over the ranks (an all-reduce of m*m + m doubles, e.g. NCCL; the paper's
 *      Server gathers whole vectors instead, Section 2, last paragraph on complexity);
 *   3. every rank calls qn_update_from_gram with the summed buffer and gets its slice of theta_new; j and
 *      sigma are the same on every rank.
 *   gram         DEVICE, m*m + m doubles as written by qn_gram (or sums of such buffers), read only
 *   other arguments as for qn_update.  Errors as for qn_update.
 * Accuracy: that of the Gram it is given.  Above 2^22 parameters (2^17 with m > 8) qn_gram rounds its products (see
 * qn_update); this call checks the spectrum against that pass's accuracy like qn_update does, but cannot repeat
 * the pass: see qn_precision_flag.
 */
QN_API qn_status qn_update_from_gram(qn_handle h, const void* theta, const void* g, const double* gram, double tau,
                                     double lambda, void* theta_new, int32_t* j_out, double* sigma_out,
                                     void* cuda_stream);

/*
 * Asynchronous mode (Section 2, first sentence: an update may follow each Write by one Worker).
 * The handle keeps a window of the m most recent (theta, g) pairs and the raw m x m Gram of the
 * window's gradients in fp64.  qn_push lands one Worker's Write in a slot and refreshes that
 * slot's Gram row and column in O(m n); the paper is silent on which pair a Write replaces:
 * slot = -1 replaces the oldest, 0 <= slot < m replaces that slot.
 *   theta_col, g_col   [n] each, read-only
 * slot = -1 moves on to the next-oldest pair only when the Write was enqueued (a call that fails on the host
 * leaves the window and its order as they were).  If a later step reports QN_ERR_DEVICE_TIMEOUT, the row refresh
 * of the most recent Write may be incomplete (its Gram row holds NaN, so every later update would report
 * QN_ERR_NONFINITE and fall back to the SGD step): push that Write again into the same slot and call qn_rebuild.
 */
QN_API qn_status qn_push(qn_handle h, int32_t slot, const void* theta_col, const void* g_col, void* cuda_stream);

/*
 * The Server step on the window's current contents.  QN_ERR_STATE until every slot has been
 * written at least once.  Outputs as in qn_update.
 * Accuracy: above 2^22 parameters the row refresh of qn_push adds fp32 products per work item before it goes to
 * fp64; measured on spectra with small retained modes, a retained sigma_k is off by about 2e-9 (sigma_1 / sigma_k)^2
 * of its value with bf16 storage and 5e-12 (sigma_1 / sigma_k)^2 with fp32 storage, whatever n: inside 1e-5 down to
 * sigma_k = 1.4e-2 sigma_1 (bf16) and 1e-3 sigma_1 (fp32).  qn_rebuild recomputes the window's Gram with fp64 products.
 */
QN_API qn_status qn_update_window(qn_handle h, double tau, double lambda, void* theta_new, int32_t* j_out,
                           double* sigma_out, void* cuda_stream);

/* Recompute the window's raw Gram from its columns in O(m^2 n) (drift correction / after restore). */
QN_API qn_status qn_rebuild(qn_handle h, void* cuda_stream);

/*
 * DEVICE pointers to the window's storage, [m][n] each, so that a caller can restore or inspect
 * it (follow a restore with qn_rebuild and qn_window_mark_full).  NULL before the first qn_push
 * unless qn_window_alloc was called.
 */
QN_API qn_status qn_window_alloc(qn_handle h);
QN_API void* qn_window_theta(qn_handle h);
QN_API void* qn_window_g(qn_handle h);
QN_API qn_status qn_window_mark_full(qn_handle h);

/*
 * qn_update with HOST buffers: copies theta and g (HOST, [m][n], pinned memory recommended) to
 * device staging owned by the handle, runs the step, copies theta_new back to theta_new_host
 * ([n]) and waits.  The staging (2 m n + n elements) is allocated by the first call.
 */
QN_API qn_status qn_update_host(qn_handle h, const void* theta_host, const void* g_host, double tau, double lambda,
                         void* theta_new_host, int32_t* j_out, double* sigma_out, void* cuda_stream);

/* Wait for the stream last used with this handle and return the deferred device status. */
QN_API qn_status qn_status_sync(qn_handle h);

/*
 * Self-test of the device-side failure reporting (the paper has no counterpart).  Every wait inside the streaming
 * kernels (on a bulk copy, a stage of the operand ring, a tensor-core commit) is bounded: when its poll limit runs
 * out the kernel stops waiting, marks its partial sums invalid, sets a device word and returns, and the next
 * eigen-solve reports QN_ERR_DEVICE_TIMEOUT.  This call enqueues a one-warp kernel that waits, with the same
 * routine, on a barrier that nothing ever arrives on (the limit is one second), and sets that word: the next step on the
 * handle then reports QN_ERR_DEVICE_TIMEOUT, and the one after it is clean again.  Nothing else is touched.
 */
QN_API qn_status qn_selftest_bounded_wait(qn_handle h, void* cuda_stream);

/* Number of kernels this handle launched in its most recent qn_* call, and since creation. */
QN_API int32_t qn_last_launches(qn_handle h);
QN_API int64_t qn_total_launches(qn_handle h);

/*
 * (The paper has no counterpart.)  Which kernel the most recent Gram pass of this handle was dispatched to (qn_update, qn_update_host, qn_gram,
 * qn_apply_hinv, qn_rebuild), or, after qn_push, which row-refresh kernel ran; QN_KERNEL_NONE before the first.
 * Benchmarks label their numbers with it.  When a step repeated its Gram pass in fp64 (see qn_update), this reports
 * the fp64 kernel once the step's results have been fetched to the host.  QN_KERNEL_FP64_PRODUCTS is or-ed in when every product and sum of the
 * pass was formed in fp64 (n below 2^22, and qn_rebuild).
 */
#define QN_KERNEL_NONE 0
#define QN_KERNEL_GRAM_DIRECT 1  /* m <= 8, register-fed, plain ALUs */
#define QN_KERNEL_GRAM_BULK 2    /* m <= 8, fed by bulk copies into shared-memory stages, packed fp32 ALUs */
#define QN_KERNEL_GRAM_TILED 3   /* 9 <= m <= 64, shared-memory tiles, plain ALUs */
#define QN_KERNEL_GRAM_TENSOR 4  /* 9 <= m <= 64, tcgen05 tensor cores, bf16 hi/lo split, fp32 chains, fp64 flush */
#define QN_KERNEL_ROW_REGISTER 5 /* row refresh, register-fed */
#define QN_KERNEL_ROW_BULK 6     /* row refresh, fed and landed by bulk copies */
#define QN_KERNEL_FP64_PRODUCTS 0x100
QN_API int32_t qn_last_gram_kernel(qn_handle h);

/*
 * (The paper has no counterpart.)  1 if the most recent step whose results were fetched to the host (j_out or sigma_out non-NULL, or qn_status_sync)
 * found a retained sigma_k too small for the accuracy of the Gram pass behind it AND could not repeat that pass
 * itself, else 0.  Only qn_update_from_gram can leave it set (qn_update, qn_update_host and qn_apply_hinv repeat
 * the pass on the device, see qn_update): the Gram it is given was summed by the caller, e.g. over the ranks of an
 * n-sharded step.  The remedy is the caller's: select QN_GRAM_PATH_FP64, call qn_gram again on every rank, sum, and
 * repeat the step (sigma and j are the same on every rank, so every rank sees the same flag).
 */
QN_API int32_t qn_precision_flag(qn_handle h);

/* Jacobi sweeps used by the most recent step whose results were fetched to the host (j_out or
 * sigma_out non-NULL, or qn_status_sync), else -1. */
QN_API int32_t qn_last_sweeps(qn_handle h);

/*
 * qn_gram without any allocation (the paper has no counterpart; this exists for deployment).
 *
 * For callers that may not allocate device memory once they are running -- code living inside a
 * framework whose caching allocator owns all of the GPU's memory, services with a no-allocation
 * rule after start-up because cudaMalloc can block, synchronise the device or fail late, plug-ins
 * that are only ever handed buffers -- and therefore cannot use qn_create.  It needs no handle:
 * the caller passes the input g ([m][n], DEVICE, as for qn_gram) and the output gram_out
 * (DEVICE, m*m + m doubles: centred Gram, then G^T gbar), and the per-CTA partial sums that the
 * pass keeps between its two kernels go to a fixed array of 716,800 bytes compiled into the
 * library, which each GPU that loads the library holds until the process exits.
 *
 * Limits: 1 <= m <= QN_STATIC_MAX_M (32); a larger m does not fit the fixed array and is rejected
 * with QN_ERR_INVALID before anything is launched.  n is unlimited.  Runs on the CURRENT device.
 * The call makes no cudaMalloc/cudaFree and calls no allocating routine; it only enqueues two
 * kernels on cuda_stream and returns.
 *
 * First call on each device: looks up the array's device address and loads every kernel variant the
 * entry point can dispatch to (whatever dtype, m, n and alignment later calls have) into the context,
 * raising their shared-memory limits; loading code may allocate device memory inside the driver.
 * Make that first call during start-up, before any stream capture; later calls of any shape load and
 * allocate nothing.
 *
 * Failure reporting: there is no handle to carry a device status.  If one of the pass's bounded device
 * waits runs out (see qn_selftest_bounded_wait), the call has already returned QN_OK and the only sign
 * is that gram_out holds NaN; non-finite input shows the same way.  Check gram_out for finiteness
 * where that matters.
 *
 * Sharing: all calls on a device use the same array, and it keeps whatever the previous call left
 * there.  Each call overwrites every entry it later reads, so nothing needs clearing and results
 * do not depend on earlier calls; but two calls whose kernels can overlap on the GPU (different
 * streams, no ordering between them) race on the array and give wrong results -- order them.
 */
#define QN_STATIC_MAX_M 32
#define QN_STATIC_MAX_CTAS 160
QN_API qn_status qn_gram_static(int64_t n, int32_t m, qn_dtype dtype, const void* g, double* gram_out,
                                void* cuda_stream);

/*
 * Per-kernel timing, for benchmarks.  Between qn_timing_begin and qn_timing_end every kernel the
 * handle launches (up to max_kernels of them) is bracketed by two CUDA events recorded on the
 * stream of the call.  qn_timing_end waits for those events and returns, per kind of kernel,
 * the summed device time in milliseconds and the number of launches:
 *   QN_TIME_GRAM     streaming Gram pass (means, centred Gram, G^T gbar; Section 2)
 *   QN_TIME_SOLVE    single-CTA partial sum, centring, Jacobi, cut-off, coefficients
 *   QN_TIME_COMBINE  streaming pass that writes theta_new (Eq. (2) with Eq. (4))
 *   QN_TIME_ROW      one-row Gram refresh of the asynchronous window
 * Timing is off by default and has no counterpart in the paper.
 */
#define QN_TIME_GRAM 0
#define QN_TIME_SOLVE 1
#define QN_TIME_COMBINE 2
#define QN_TIME_ROW 3
#define QN_TIME_KINDS 4
QN_API qn_status qn_timing_begin(qn_handle h, int32_t max_kernels);
QN_API qn_status qn_timing_end(qn_handle h, double ms_total[QN_TIME_KINDS], int32_t count[QN_TIME_KINDS]);

#ifdef __cplusplus
}
#endif
#endif /* QN_H */
