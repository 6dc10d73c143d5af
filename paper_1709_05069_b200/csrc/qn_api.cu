// C ABI of libqn: argument checks, workspace, launch sequences.  See include/qn.h for the contract.
#include <math.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include <nvtx3/nvToolsExt.h>

#include "qn_internal.h"

struct qn_ctx {
    int64_t n;
    int32_t m;
    qn_dtype dtype;
    size_t elem;
    int device;

    double* partials;  // device, max_partials * qn_partial_len(m)
    int max_partials;
    qn_coef_block* coef;          // device
    qn_result_block* result;      // device
    qn_result_block* host_result; // pinned host
    unsigned int* ticket;         // device, zero between launches
    int* error_word;              // device, set by a kernel that gave up on a bounded wait
    double* rhs;                  // device, m doubles: g_k^T z of qn_apply_hinv
    int32_t j_cap;                // < 0: none
    int32_t sweep_limit;          // limit on the fp64 Jacobi sweeps, 0 = the built-in one
    int32_t gram_path;            // QN_GRAM_PATH_* (qn_set_gram_path)
    int32_t tau_cap;              // learning-rate cap on/off (qn_update and qn_update_host)
    double* partials_theta;       // device, as `partials`, allocated when the cap is first switched on
    double last_tau;              // learning rate of the most recent step whose results were fetched

    // asynchronous window
    void* win_theta;
    void* win_g;
    double* raw_gram;  // device, m*m
    uint64_t filled;   // bit k set once slot k has been written
    int32_t head;      // slot of the oldest column

    // host-buffer path
    void* stage_theta;
    void* stage_g;
    void* stage_out;
    cudaStream_t copy_stream;     // carries theta's host-to-device copy while the Gram pass runs
    cudaEvent_t ev_fork, ev_theta;

    // optional per-kernel timing with CUDA events on the launching stream
    cudaEvent_t* ev;       // 2 events per timed kernel
    int32_t* ev_kind;
    int32_t ev_cap, ev_used;

    cudaStream_t last_stream;
    int32_t last_launches;
    int64_t total_launches;
    int32_t last_sweeps;
    int32_t last_kernel;  // QN_KERNEL_* of the most recent Gram or row pass
    int32_t redo_kernel;  // QN_KERNEL_* of the fp64 repeat pass that the most recent step enqueued (0: none)
    int32_t gram_call_kernel;  // QN_KERNEL_* of the most recent qn_gram call on this handle (0: none yet)
    int32_t precision_flag;    // bit 0 of the result block's redo word as last fetched
};

static int g_sm_count_cache[64];

int qn_sm_count() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 1;
    if (dev >= 0 && dev < 64 && g_sm_count_cache[dev] > 0) return g_sm_count_cache[dev];
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) sms = 1;
    if (dev >= 0 && dev < 64) g_sm_count_cache[dev] = sms;
    return sms;
}

extern "C" const char* qn_strerror(qn_status s) {
    switch (s) {
        case QN_OK: return "ok";
        case QN_ERR_INVALID: return "invalid argument";
        case QN_ERR_ALLOC: return "allocation failed";
        case QN_ERR_CUDA: return "CUDA runtime error";
        case QN_ERR_STATE: return "call not valid in this state";
        case QN_ERR_NOT_CONVERGED: return "Jacobi sweep limit reached";
        case QN_ERR_NONFINITE: return "non-finite Gram";
        case QN_ERR_DEVICE_TIMEOUT: return "device wait limit reached";
    }
    return "unknown status";
}

namespace {

struct DeviceGuard {
    int prev = -1;
    bool ok = false;
    explicit DeviceGuard(int dev) {
        if (cudaGetDevice(&prev) != cudaSuccess) return;
        ok = (prev == dev) || cudaSetDevice(dev) == cudaSuccess;
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

inline bool finite_d(double x) { return isfinite(x); }

// Brackets one kernel launch with an NVTX range (visible to a profiler, free without one) and, when timing is on
// (see qn_timing_begin), with two events.
struct KernelTimer {
    qn_handle h;
    cudaStream_t st;
    int idx = -1;
    KernelTimer(qn_handle h_, cudaStream_t st_, int kind) : h(h_), st(st_) {
        static const char* const names[QN_TIME_KINDS] = {"qn:gram", "qn:solve", "qn:combine", "qn:row"};
        nvtxRangePushA(names[kind]);
        if (h->ev && h->ev_used < h->ev_cap) {
            idx = h->ev_used++;
            h->ev_kind[idx] = kind;
            cudaEventRecord(h->ev[2 * idx], st);
        }
    }
    ~KernelTimer() {
        if (idx >= 0) cudaEventRecord(h->ev[2 * idx + 1], st);
        nvtxRangePop();
    }
};

inline void begin_call(qn_handle h, cudaStream_t st) {
    h->last_launches = 0;
    h->last_stream = st;
}

inline void end_call(qn_handle h) { h->total_launches += h->last_launches; }

// Bring the result block to the host (waits for the stream) and hand j / sigma to the caller.
qn_status fetch_result(qn_handle h, cudaStream_t st, int32_t* j_out, double* sigma_out) {
    if (cudaMemcpyAsync(h->host_result, h->result, sizeof(qn_result_block), cudaMemcpyDeviceToHost, st) != cudaSuccess)
        return QN_ERR_CUDA;
    if (cudaStreamSynchronize(st) != cudaSuccess) return QN_ERR_CUDA;
    if (j_out) *j_out = h->host_result->j;
    if (sigma_out) memcpy(sigma_out, h->host_result->sigma, sizeof(double) * h->m);
    h->last_sweeps = h->host_result->sweeps;
    h->last_tau = h->host_result->tau_eff;
    if ((h->host_result->redo & 2) && h->redo_kernel) h->last_kernel = h->redo_kernel;  // the fp64 repeat pass ran
    h->precision_flag = h->host_result->redo & 1;
    return static_cast<qn_status>(h->host_result->status);
}

qn_status check_step_args(qn_handle h, double tau, double lambda, const void* theta_new) {
    if (!h || !theta_new) return QN_ERR_INVALID;
    if (!finite_d(tau) || !finite_d(lambda) || !(lambda > 0.0)) return QN_ERR_INVALID;
    return QN_OK;
}

// A pointer the kernels of this handle may dereference: device memory of the handle's device, or managed memory.
// Anything else (host memory, another GPU's memory) would fault on the device, so it is refused on the host.
bool on_device(const void* p, int dev) {
    cudaPointerAttributes a;
    if (cudaPointerGetAttributes(&a, p) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    if (a.type == cudaMemoryTypeManaged) return true;
    return a.type == cudaMemoryTypeDevice && a.device == dev;
}

bool overlaps(const void* a, size_t na, const void* b, size_t nb) {
    const uintptr_t a0 = reinterpret_cast<uintptr_t>(a), b0 = reinterpret_cast<uintptr_t>(b);
    return a0 < b0 + nb && b0 < a0 + na;
}

// After the first solve of a step whose Gram pass had reduced precision: the same pass with every product in fp64,
// and a second solve.  Both kernels return at once unless the first solve found a retained sigma_k so small that the
// reduced-precision pass cannot deliver it to 1e-5 (result->redo, on the device: the host does not wait to find out).
qn_status precise_redo(qn_handle h, const void* g, qn_solve_params p, double lambda, cudaStream_t st) {
    h->redo_kernel = 0;
    p.redo_coeff = qn_gram_error_coeff(h->last_kernel, h->dtype, h->n, lambda);
    if (!(p.redo_coeff > 0.0)) return QN_OK;
    // every retained sigma_k is at least lambda sigma_1: with this lambda the first solve cannot ask for a repeat
    if (lambda >= 1.0 || p.redo_coeff / (lambda * lambda) <= QN_REDO_TRIGGER) return QN_OK;
    const int* run_if = &h->result->redo;  // device address; not dereferenced here
    int np = 0;
    {
        KernelTimer t(h, st, QN_TIME_GRAM);
        if (qn_launch_gram(h->dtype, g, h->n, h->m, false, h->partials, &np, h->max_partials, st, &h->last_launches,
                           h->error_word, lambda, QN_GRAM_PATH_FP64, &h->redo_kernel, run_if) != cudaSuccess)
            return QN_ERR_CUDA;
    }
    p.num_partials = np;
    p.only_if_redo = 1;
    p.redo_coeff = 0.0;
    KernelTimer t(h, st, QN_TIME_SOLVE);
    return qn_launch_solve(p, st, &h->last_launches) == cudaSuccess ? QN_OK : QN_ERR_CUDA;
}

// Gram partials -> solve -> combine on device buffers.
// theta_ready (may be NULL): an event the stream waits for before the first kernel that reads theta.
qn_status run_step(qn_handle h, const void* theta, const void* g, double tau, double lambda, void* theta_new,
                   cudaStream_t st, cudaEvent_t theta_ready = nullptr) {
    int np = 0;
    {
        KernelTimer t(h, st, QN_TIME_GRAM);
        if (qn_launch_gram(h->dtype, g, h->n, h->m, false, h->partials, &np, h->max_partials, st,
                           &h->last_launches, h->error_word, lambda, h->gram_path, &h->last_kernel) != cudaSuccess)
            return QN_ERR_CUDA;
    }
    int np_theta = 0;
    if (h->tau_cap && h->partials_theta) {
        // the learning-rate cap needs ||Theta v_k||: one more Gram pass, over theta
        if (theta_ready) {
            if (cudaStreamWaitEvent(st, theta_ready, 0) != cudaSuccess) return QN_ERR_CUDA;
            theta_ready = nullptr;
        }
        KernelTimer t(h, st, QN_TIME_GRAM);
        if (qn_launch_gram(h->dtype, theta, h->n, h->m, false, h->partials_theta, &np_theta, h->max_partials, st,
                           &h->last_launches, h->error_word, lambda, h->gram_path) != cudaSuccess)
            return QN_ERR_CUDA;
    }
    qn_solve_params p;
    memset(&p, 0, sizeof(p));
    p.j_cap = h->j_cap;
    p.max_sweeps = h->sweep_limit;
    p.tau_cap = h->tau_cap && h->partials_theta;
    p.partials_theta = h->partials_theta;
    p.num_partials_theta = np_theta;
    p.m = h->m;
    p.source = QN_SRC_PARTIALS;
    p.partials = h->partials;
    p.num_partials = np;
    p.tau = tau;
    p.lambda = lambda;
    p.coef = h->coef;
    p.result = h->result;
    p.error_word = h->error_word;
    p.redo_coeff = qn_gram_error_coeff(h->last_kernel, h->dtype, h->n, lambda);
    {
        KernelTimer t(h, st, QN_TIME_SOLVE);
        if (qn_launch_solve(p, st, &h->last_launches) != cudaSuccess) return QN_ERR_CUDA;
    }
    if (precise_redo(h, g, p, lambda, st) != QN_OK) return QN_ERR_CUDA;
    if (theta_ready && cudaStreamWaitEvent(st, theta_ready, 0) != cudaSuccess) return QN_ERR_CUDA;
    {
        KernelTimer t(h, st, QN_TIME_COMBINE);
        if (qn_launch_combine(h->dtype, theta, g, h->n, h->m, h->coef, theta_new, st, &h->last_launches) !=
            cudaSuccess)
            return QN_ERR_CUDA;
    }
    return QN_OK;
}

qn_status ensure_window(qn_handle h) {
    if (h->win_theta) return QN_OK;
    const size_t bytes = (size_t)h->m * (size_t)h->n * h->elem;
    void *a = nullptr, *b = nullptr;
    if (cudaMalloc(&a, bytes) != cudaSuccess) {
        cudaGetLastError();
        return QN_ERR_ALLOC;
    }
    if (cudaMalloc(&b, bytes) != cudaSuccess) {
        cudaGetLastError();
        cudaFree(a);
        return QN_ERR_ALLOC;
    }
    h->win_theta = a;
    h->win_g = b;
    h->filled = 0;
    h->head = 0;
    return QN_OK;
}

}  // namespace

extern "C" qn_status qn_create(int64_t n, int32_t m, qn_dtype dtype, qn_handle* out) {
    if (!out || n < 1 || m < 1 || m > QN_MAX_M || (dtype != QN_F32 && dtype != QN_BF16)) return QN_ERR_INVALID;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) {
        cudaGetLastError();
        return QN_ERR_CUDA;
    }
    if (qn_solve_init() != cudaSuccess) {
        cudaGetLastError();
        return QN_ERR_CUDA;
    }
    qn_ctx* h = new (std::nothrow) qn_ctx();
    if (!h) return QN_ERR_ALLOC;
    memset(h, 0, sizeof(*h));
    h->n = n;
    h->m = m;
    h->dtype = dtype;
    h->elem = dtype == QN_F32 ? 4 : 2;
    h->device = dev;
    h->last_sweeps = -1;
    h->j_cap = -1;
    h->max_partials = qn_sm_count() * 4;
    bool ok = cudaMalloc(&h->partials, sizeof(double) * (size_t)h->max_partials * qn_partial_len(m)) == cudaSuccess;
    ok = ok && cudaMalloc(&h->coef, sizeof(qn_coef_block)) == cudaSuccess;
    ok = ok && cudaMalloc(&h->result, sizeof(qn_result_block)) == cudaSuccess;
    ok = ok && cudaMalloc(&h->raw_gram, sizeof(double) * m * m) == cudaSuccess;
    ok = ok && cudaMalloc(&h->ticket, sizeof(unsigned int)) == cudaSuccess;
    ok = ok && cudaMalloc(&h->rhs, sizeof(double) * QN_MAX_M) == cudaSuccess;
    ok = ok && cudaMalloc(&h->error_word, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMemset(h->error_word, 0, sizeof(int)) == cudaSuccess;
    ok = ok && cudaMallocHost(&h->host_result, sizeof(qn_result_block)) == cudaSuccess;
    ok = ok && cudaMemset(h->ticket, 0, sizeof(unsigned int)) == cudaSuccess;
    ok = ok && cudaMemset(h->result, 0, sizeof(qn_result_block)) == cudaSuccess;
    ok = ok && cudaMemset(h->raw_gram, 0, sizeof(double) * m * m) == cudaSuccess;
    if (!ok) {
        cudaGetLastError();
        qn_destroy(h);
        return QN_ERR_ALLOC;
    }
    *out = h;
    return QN_OK;
}

extern "C" qn_status qn_destroy(qn_handle h) {
    if (!h) return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    cudaDeviceSynchronize();
    cudaFree(h->partials);
    cudaFree(h->coef);
    cudaFree(h->result);
    cudaFree(h->raw_gram);
    cudaFree(h->ticket);
    cudaFree(h->rhs);
    cudaFree(h->partials_theta);
    cudaFree(h->error_word);
    cudaFree(h->win_theta);
    cudaFree(h->win_g);
    cudaFree(h->stage_theta);
    cudaFree(h->stage_g);
    cudaFree(h->stage_out);
    if (h->host_result) cudaFreeHost(h->host_result);
    if (h->copy_stream) {
        cudaStreamDestroy(h->copy_stream);
        cudaEventDestroy(h->ev_fork);
        cudaEventDestroy(h->ev_theta);
    }
    if (h->ev) {
        for (int i = 0; i < 2 * h->ev_cap; ++i) cudaEventDestroy(h->ev[i]);
        free(h->ev);
        free(h->ev_kind);
    }
    cudaGetLastError();
    delete h;
    return QN_OK;
}

extern "C" qn_status qn_set_tau_cap(qn_handle h, int32_t on) {
    if (!h) return QN_ERR_INVALID;
    if (on && !h->partials_theta) {
        DeviceGuard guard(h->device);
        if (!guard.ok) return QN_ERR_CUDA;
        if (cudaMalloc(&h->partials_theta, sizeof(double) * (size_t)h->max_partials * qn_partial_len(h->m)) !=
            cudaSuccess) {
            cudaGetLastError();
            h->partials_theta = nullptr;
            return QN_ERR_ALLOC;
        }
    }
    h->tau_cap = on ? 1 : 0;
    return QN_OK;
}

extern "C" double qn_last_tau(qn_handle h) { return h ? h->last_tau : 0.0; }

extern "C" qn_status qn_set_rank_cap(qn_handle h, int32_t j_cap) {
    if (!h) return QN_ERR_INVALID;
    h->j_cap = j_cap < 0 ? -1 : j_cap;
    return QN_OK;
}

extern "C" qn_status qn_set_sweep_limit(qn_handle h, int32_t max_sweeps) {
    if (!h || max_sweeps < 0) return QN_ERR_INVALID;
    h->sweep_limit = max_sweeps;
    return QN_OK;
}

extern "C" qn_status qn_set_gram_path(qn_handle h, int32_t path) {
    if (!h || (path != QN_GRAM_PATH_AUTO && path != QN_GRAM_PATH_PLAIN_ALU && path != QN_GRAM_PATH_FP64))
        return QN_ERR_INVALID;
    h->gram_path = path;
    return QN_OK;
}

extern "C" qn_status qn_update(qn_handle h, const void* theta, const void* g, double tau, double lambda,
                               void* theta_new, int32_t* j_out, double* sigma_out, void* cuda_stream) {
    qn_status s = check_step_args(h, tau, lambda, theta_new);
    if (s != QN_OK) return s;
    if (!theta || !g) return QN_ERR_INVALID;
    const size_t in_bytes = (size_t)h->m * (size_t)h->n * h->elem, out_bytes = (size_t)h->n * h->elem;
    if (overlaps(theta_new, out_bytes, theta, in_bytes) || overlaps(theta_new, out_bytes, g, in_bytes))
        return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    if (!on_device(theta, h->device) || !on_device(g, h->device) || !on_device(theta_new, h->device))
        return QN_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    begin_call(h, st);
    s = run_step(h, theta, g, tau, lambda, theta_new, st);
    end_call(h);
    if (s != QN_OK) return s;
    if (j_out || sigma_out) return fetch_result(h, st, j_out, sigma_out);
    return QN_OK;
}

extern "C" qn_status qn_update_from_gram(qn_handle h, const void* theta, const void* g, const double* gram,
                                         double tau, double lambda, void* theta_new, int32_t* j_out,
                                         double* sigma_out, void* cuda_stream) {
    qn_status s = check_step_args(h, tau, lambda, theta_new);
    if (s != QN_OK) return s;
    if (!theta || !g || !gram) return QN_ERR_INVALID;
    const size_t in_bytes = (size_t)h->m * (size_t)h->n * h->elem, out_bytes = (size_t)h->n * h->elem;
    if (overlaps(theta_new, out_bytes, theta, in_bytes) || overlaps(theta_new, out_bytes, g, in_bytes))
        return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    if (!on_device(theta, h->device) || !on_device(g, h->device) || !on_device(theta_new, h->device) ||
        !on_device(gram, h->device))
        return QN_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    begin_call(h, st);
    qn_solve_params p;
    memset(&p, 0, sizeof(p));
    p.j_cap = h->j_cap;
    p.max_sweeps = h->sweep_limit;
    p.m = h->m;
    p.source = QN_SRC_SUMMED;
    p.raw_gram = const_cast<double*>(gram);  // read only in this mode
    // If this handle's qn_gram produced the buffer (the n-sharded step), the solve can still judge the spectrum against
    // that pass's accuracy; it cannot repeat the pass (the sum over the ranks is the caller's), so it only raises the
    // flag that qn_precision_flag returns.
    p.redo_coeff = h->gram_call_kernel ? qn_gram_error_coeff(h->gram_call_kernel, h->dtype, h->n, lambda) : 0.0;
    p.tau = tau;
    p.lambda = lambda;
    p.coef = h->coef;
    p.result = h->result;
    p.error_word = h->error_word;
    {
        KernelTimer t(h, st, QN_TIME_SOLVE);
        if (qn_launch_solve(p, st, &h->last_launches) != cudaSuccess) s = QN_ERR_CUDA;
    }
    if (s == QN_OK) {
        KernelTimer t(h, st, QN_TIME_COMBINE);
        if (qn_launch_combine(h->dtype, theta, g, h->n, h->m, h->coef, theta_new, st, &h->last_launches) !=
            cudaSuccess)
            s = QN_ERR_CUDA;
    }
    end_call(h);
    if (s != QN_OK) return s;
    if (j_out || sigma_out) return fetch_result(h, st, j_out, sigma_out);
    return QN_OK;
}

extern "C" qn_status qn_apply_hinv(qn_handle h, const void* theta, const void* g, double lambda, const void* z,
                                   void* out, int32_t* j_out, double* sigma_out, void* cuda_stream) {
    qn_status s = check_step_args(h, 1.0, lambda, out);
    if (s != QN_OK) return s;
    if (!theta || !g || !z) return QN_ERR_INVALID;
    const size_t in_bytes = (size_t)h->m * (size_t)h->n * h->elem, vec_bytes = (size_t)h->n * h->elem;
    if (overlaps(out, vec_bytes, theta, in_bytes) || overlaps(out, vec_bytes, g, in_bytes) ||
        overlaps(out, vec_bytes, z, vec_bytes))
        return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    if (!on_device(theta, h->device) || !on_device(g, h->device) || !on_device(z, h->device) ||
        !on_device(out, h->device))
        return QN_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    begin_call(h, st);
    // 1. g_k^T z for every Worker (the row pass of the asynchronous mode with z in the place of the new column;
    //    it uses the partials buffer as scratch, so it comes before the Gram pass)
    bool landed = false;
    {
        KernelTimer t(h, st, QN_TIME_ROW);
        if (qn_launch_row(h->dtype, g, z, nullptr, nullptr, nullptr, h->n, h->m, -1, h->partials, h->max_partials,
                          nullptr, h->rhs, h->ticket, h->error_word, &landed, st, &h->last_launches) != cudaSuccess)
            s = QN_ERR_CUDA;
    }
    // 2. Gram pass, 3. eigen-solve with the coefficients built for z, 4. out = z - G d + Theta d
    int np = 0;
    if (s == QN_OK) {
        KernelTimer t(h, st, QN_TIME_GRAM);
        if (qn_launch_gram(h->dtype, g, h->n, h->m, false, h->partials, &np, h->max_partials, st, &h->last_launches,
                           h->error_word, lambda, h->gram_path, &h->last_kernel) != cudaSuccess)
            s = QN_ERR_CUDA;
    }
    if (s == QN_OK) {
        qn_solve_params p;
        memset(&p, 0, sizeof(p));
        p.j_cap = h->j_cap;
        p.max_sweeps = h->sweep_limit;
        p.m = h->m;
        p.source = QN_SRC_PARTIALS;
        p.partials = h->partials;
        p.num_partials = np;
        p.rhs_raw = h->rhs;
        p.tau = -1.0;
        p.lambda = lambda;
        p.coef = h->coef;
        p.result = h->result;
        p.error_word = h->error_word;
        p.redo_coeff = qn_gram_error_coeff(h->last_kernel, h->dtype, h->n, lambda);
        {
            KernelTimer t(h, st, QN_TIME_SOLVE);
            if (qn_launch_solve(p, st, &h->last_launches) != cudaSuccess) s = QN_ERR_CUDA;
        }
        if (s == QN_OK) s = precise_redo(h, g, p, lambda, st);
    }
    if (s == QN_OK) {
        KernelTimer t(h, st, QN_TIME_COMBINE);
        if (qn_launch_combine(h->dtype, theta, g, h->n, h->m, h->coef, out, st, &h->last_launches, z) != cudaSuccess)
            s = QN_ERR_CUDA;
    }
    end_call(h);
    if (s != QN_OK) return s;
    if (j_out || sigma_out) return fetch_result(h, st, j_out, sigma_out);
    return QN_OK;
}

extern "C" qn_status qn_gram(qn_handle h, const void* g, double* gram_out, void* cuda_stream) {
    if (!h || !g || !gram_out) return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    if (!on_device(g, h->device) || !on_device(gram_out, h->device)) return QN_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    begin_call(h, st);
    int np = 0;
    qn_status s = QN_OK;
    {
        KernelTimer t(h, st, QN_TIME_GRAM);
        if (qn_launch_gram(h->dtype, g, h->n, h->m, false, h->partials, &np, h->max_partials, st, &h->last_launches,
                           h->error_word, 0.0, h->gram_path, &h->last_kernel) != cudaSuccess)
            s = QN_ERR_CUDA;
    }
    if (s == QN_OK) {
        qn_solve_params p;
        memset(&p, 0, sizeof(p));
        p.j_cap = h->j_cap;
        p.max_sweeps = h->sweep_limit;
        p.m = h->m;
        p.source = QN_SRC_PARTIALS;
        p.partials = h->partials;
        p.num_partials = np;
        p.error_word = h->error_word;
        p.gram_out = gram_out;
        p.gram_only = 1;
        p.lambda = 1.0;
        p.coef = h->coef;
        p.result = h->result;
        h->gram_call_kernel = h->last_kernel;
        KernelTimer t(h, st, QN_TIME_SOLVE);
        if (qn_launch_solve(p, st, &h->last_launches) != cudaSuccess) s = QN_ERR_CUDA;
    }
    end_call(h);
    return s;
}

extern "C" qn_status qn_window_alloc(qn_handle h) {
    if (!h) return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    return ensure_window(h);
}

extern "C" void* qn_window_theta(qn_handle h) { return h ? h->win_theta : nullptr; }
extern "C" void* qn_window_g(qn_handle h) { return h ? h->win_g : nullptr; }

extern "C" qn_status qn_window_mark_full(qn_handle h) {
    if (!h) return QN_ERR_INVALID;
    if (!h->win_theta) return QN_ERR_STATE;
    h->filled = h->m == 64 ? ~0ull : ((1ull << h->m) - 1ull);
    return QN_OK;
}

extern "C" qn_status qn_push(qn_handle h, int32_t slot, const void* theta_col, const void* g_col, void* cuda_stream) {
    if (!h || !theta_col || !g_col || slot < -1 || slot >= h->m) return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    if (!on_device(theta_col, h->device) || !on_device(g_col, h->device)) return QN_ERR_INVALID;
    qn_status s = ensure_window(h);
    if (s != QN_OK) return s;
    const size_t col_bytes = (size_t)h->n * h->elem, win_bytes = col_bytes * h->m;
    if (overlaps(theta_col, col_bytes, h->win_theta, win_bytes) || overlaps(g_col, col_bytes, h->win_g, win_bytes))
        return QN_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    begin_call(h, st);
    const bool oldest = slot < 0;
    if (oldest) slot = h->head;
    char* trow = static_cast<char*>(h->win_theta) + (size_t)slot * col_bytes;
    char* grow = static_cast<char*>(h->win_g) + (size_t)slot * col_bytes;
    bool theta_landed = false;
    {
        KernelTimer t(h, st, QN_TIME_ROW);
        if (qn_launch_row(h->dtype, h->win_g, g_col, grow, theta_col, trow, h->n, h->m, slot, h->partials,
                          h->max_partials, h->raw_gram, nullptr, h->ticket, h->error_word, &theta_landed, st,
                          &h->last_launches) != cudaSuccess)
            s = QN_ERR_CUDA;
    }
    // the register kernel lands only the gradient column
    if (s == QN_OK && !theta_landed &&
        cudaMemcpyAsync(trow, theta_col, col_bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        s = QN_ERR_CUDA;
    if (s == QN_OK) {
        h->last_kernel = (theta_landed ? QN_KERNEL_ROW_BULK : QN_KERNEL_ROW_REGISTER) |
                         (h->n < QN_PRECISE_BELOW ? QN_KERNEL_FP64_PRODUCTS : 0);
        h->filled |= (1ull << slot);
        if (oldest) h->head = (h->head + 1) % h->m;  // a Write that could not be enqueued does not use up its slot
    }
    end_call(h);
    return s;
}

extern "C" qn_status qn_update_window(qn_handle h, double tau, double lambda, void* theta_new, int32_t* j_out,
                                      double* sigma_out, void* cuda_stream) {
    qn_status s = check_step_args(h, tau, lambda, theta_new);
    if (s != QN_OK) return s;
    const uint64_t full = h->m == 64 ? ~0ull : ((1ull << h->m) - 1ull);
    if (!h->win_theta || h->filled != full) return QN_ERR_STATE;
    const size_t win_bytes = (size_t)h->m * (size_t)h->n * h->elem, out_bytes = (size_t)h->n * h->elem;
    if (overlaps(theta_new, out_bytes, h->win_theta, win_bytes) || overlaps(theta_new, out_bytes, h->win_g, win_bytes))
        return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    if (!on_device(theta_new, h->device)) return QN_ERR_INVALID;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    begin_call(h, st);
    qn_solve_params p;
    memset(&p, 0, sizeof(p));
    p.j_cap = h->j_cap;
    p.max_sweeps = h->sweep_limit;
    p.m = h->m;
    p.source = QN_SRC_WINDOW;
    p.raw_gram = h->raw_gram;
    p.error_word = h->error_word;
    p.tau = tau;
    p.lambda = lambda;
    p.coef = h->coef;
    p.result = h->result;
    {
        KernelTimer t(h, st, QN_TIME_SOLVE);
        if (qn_launch_solve(p, st, &h->last_launches) != cudaSuccess) s = QN_ERR_CUDA;
    }
    if (s == QN_OK) {
        KernelTimer t(h, st, QN_TIME_COMBINE);
        if (qn_launch_combine(h->dtype, h->win_theta, h->win_g, h->n, h->m, h->coef, theta_new, st,
                              &h->last_launches) != cudaSuccess)
            s = QN_ERR_CUDA;
    }
    end_call(h);
    if (s != QN_OK) return s;
    if (j_out || sigma_out) return fetch_result(h, st, j_out, sigma_out);
    return QN_OK;
}

extern "C" qn_status qn_rebuild(qn_handle h, void* cuda_stream) {
    if (!h) return QN_ERR_INVALID;
    if (!h->win_theta) return QN_ERR_STATE;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    begin_call(h, st);
    int np = 0;
    qn_status s = QN_OK;
    if (qn_launch_gram(h->dtype, h->win_g, h->n, h->m, true, h->partials, &np, h->max_partials, st,
                       &h->last_launches, nullptr, 0.0, QN_GRAM_PATH_AUTO, &h->last_kernel) != cudaSuccess)
        s = QN_ERR_CUDA;
    if (s == QN_OK) {
        qn_solve_params p;
        memset(&p, 0, sizeof(p));
        p.j_cap = h->j_cap;
        p.max_sweeps = h->sweep_limit;
        p.m = h->m;
        p.source = QN_SRC_PARTIALS;
        p.partials = h->partials;
        p.num_partials = np;
        p.raw_gram = h->raw_gram;
        p.gram_only = 1;
        p.lambda = 1.0;
        p.coef = h->coef;
        p.result = h->result;
        if (qn_launch_solve(p, st, &h->last_launches) != cudaSuccess) s = QN_ERR_CUDA;
    }
    end_call(h);
    return s;
}

extern "C" qn_status qn_update_host(qn_handle h, const void* theta_host, const void* g_host, double tau, double lambda,
                                    void* theta_new_host, int32_t* j_out, double* sigma_out, void* cuda_stream) {
    qn_status s = check_step_args(h, tau, lambda, theta_new_host);
    if (s != QN_OK) return s;
    if (!theta_host || !g_host) return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    const size_t in_bytes = (size_t)h->m * (size_t)h->n * h->elem, out_bytes = (size_t)h->n * h->elem;
    if (!h->stage_theta) {
        bool ok = cudaMalloc(&h->stage_theta, in_bytes) == cudaSuccess;
        ok = ok && cudaMalloc(&h->stage_g, in_bytes) == cudaSuccess;
        ok = ok && cudaMalloc(&h->stage_out, out_bytes) == cudaSuccess;
        if (!ok) {
            cudaGetLastError();
            cudaFree(h->stage_theta);
            cudaFree(h->stage_g);
            cudaFree(h->stage_out);
            h->stage_theta = h->stage_g = h->stage_out = nullptr;
            return QN_ERR_ALLOC;
        }
    }
    if (!h->copy_stream) {
        cudaStream_t cs = nullptr;
        cudaEvent_t e0 = nullptr, e1 = nullptr;
        bool ok = cudaStreamCreateWithFlags(&cs, cudaStreamNonBlocking) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&e0, cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&e1, cudaEventDisableTiming) == cudaSuccess;
        if (!ok) {  // leave the handle as it was
            if (e1) cudaEventDestroy(e1);
            if (e0) cudaEventDestroy(e0);
            if (cs) cudaStreamDestroy(cs);
            cudaGetLastError();
            return QN_ERR_CUDA;
        }
        h->copy_stream = cs;
        h->ev_fork = e0;
        h->ev_theta = e1;
    }
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    begin_call(h, st);
    // g goes first on the caller's stream, since the Gram pass and the eigen-solve need only g.  theta's copy is
    // enqueued on a second stream (ordered after the work already on the caller's stream: the staging may still be
    // read by an earlier step), so it runs behind g's copy on the link and overlaps the Gram pass and the solve; the
    // caller's stream waits for it just before the pass that reads theta.
    if (cudaMemcpyAsync(h->stage_g, g_host, in_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) s = QN_ERR_CUDA;
    if (s == QN_OK && (cudaEventRecord(h->ev_fork, st) != cudaSuccess ||
                       cudaStreamWaitEvent(h->copy_stream, h->ev_fork, 0) != cudaSuccess ||
                       cudaMemcpyAsync(h->stage_theta, theta_host, in_bytes, cudaMemcpyHostToDevice, h->copy_stream) !=
                           cudaSuccess ||
                       cudaEventRecord(h->ev_theta, h->copy_stream) != cudaSuccess))
        s = QN_ERR_CUDA;
    if (s == QN_OK) s = run_step(h, h->stage_theta, h->stage_g, tau, lambda, h->stage_out, st, h->ev_theta);
    if (s == QN_OK &&
        cudaMemcpyAsync(theta_new_host, h->stage_out, out_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
        s = QN_ERR_CUDA;
    end_call(h);
    if (s != QN_OK) return s;
    return fetch_result(h, st, j_out, sigma_out);
}

extern "C" qn_status qn_status_sync(qn_handle h) {
    if (!h) return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    return fetch_result(h, h->last_stream, nullptr, nullptr);
}

extern "C" qn_status qn_selftest_bounded_wait(qn_handle h, void* cuda_stream) {
    if (!h) return QN_ERR_INVALID;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    return qn_launch_wait_probe(h->error_word, static_cast<cudaStream_t>(cuda_stream)) == cudaSuccess ? QN_OK : QN_ERR_CUDA;
}

extern "C" int32_t qn_last_launches(qn_handle h) { return h ? h->last_launches : 0; }
extern "C" int64_t qn_total_launches(qn_handle h) { return h ? h->total_launches : 0; }
extern "C" int32_t qn_last_sweeps(qn_handle h) { return h ? h->last_sweeps : -1; }
extern "C" int32_t qn_last_gram_kernel(qn_handle h) { return h ? h->last_kernel : QN_KERNEL_NONE; }
extern "C" int32_t qn_precision_flag(qn_handle h) { return h ? h->precision_flag : 0; }

extern "C" qn_status qn_timing_begin(qn_handle h, int32_t max_kernels) {
    if (!h || max_kernels < 1 || max_kernels > (1 << 20)) return QN_ERR_INVALID;
    if (h->ev) return QN_ERR_STATE;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    cudaEvent_t* ev = static_cast<cudaEvent_t*>(calloc((size_t)2 * max_kernels, sizeof(cudaEvent_t)));
    int32_t* kind = static_cast<int32_t*>(calloc((size_t)max_kernels, sizeof(int32_t)));
    if (!ev || !kind) {
        free(ev);
        free(kind);
        return QN_ERR_ALLOC;
    }
    for (int i = 0; i < 2 * max_kernels; ++i) {
        if (cudaEventCreate(&ev[i]) != cudaSuccess) {
            for (int k = 0; k < i; ++k) cudaEventDestroy(ev[k]);
            free(ev);
            free(kind);
            cudaGetLastError();
            return QN_ERR_CUDA;
        }
    }
    h->ev_kind = kind;
    h->ev_cap = max_kernels;
    h->ev_used = 0;
    h->ev = ev;
    return QN_OK;
}

extern "C" qn_status qn_timing_end(qn_handle h, double ms_total[QN_TIME_KINDS], int32_t count[QN_TIME_KINDS]) {
    if (!h || !ms_total || !count) return QN_ERR_INVALID;
    if (!h->ev) return QN_ERR_STATE;
    DeviceGuard guard(h->device);
    if (!guard.ok) return QN_ERR_CUDA;
    qn_status s = QN_OK;
    for (int k = 0; k < QN_TIME_KINDS; ++k) {
        ms_total[k] = 0.0;
        count[k] = 0;
    }
    for (int i = 0; i < h->ev_used && s == QN_OK; ++i) {
        float ms = 0.f;
        if (cudaEventSynchronize(h->ev[2 * i + 1]) != cudaSuccess ||
            cudaEventElapsedTime(&ms, h->ev[2 * i], h->ev[2 * i + 1]) != cudaSuccess) {
            s = QN_ERR_CUDA;
            break;
        }
        ms_total[h->ev_kind[i]] += ms;
        count[h->ev_kind[i]] += 1;
    }
    for (int i = 0; i < 2 * h->ev_cap; ++i) cudaEventDestroy(h->ev[i]);
    free(h->ev);
    free(h->ev_kind);
    h->ev = nullptr;
    h->ev_kind = nullptr;
    h->ev_cap = h->ev_used = 0;
    cudaGetLastError();
    return s;
}
