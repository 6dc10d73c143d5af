// qn_gram_static: the Gram reductions of qn_gram for callers that must not allocate.
//
// Some users of this library run where device allocation is off the table: inside a training loop
// whose memory is owned entirely by a caching allocator, under a real-time or safety budget that
// forbids cudaMalloc after start-up (it can block, synchronise the device or fail late), or in a
// plug-in that is only handed buffers.  Creating a qn_handle allocates; this entry point does not.
// The per-CTA partial sums that the streaming Gram pass needs between its two kernels live in the
// file-scope device array below, which every GPU that loads the library holds until the process
// exits.
#include <string.h>

#include "qn_internal.h"

// 160 CTAs x (32*33/2 + 32) doubles = 716,800 bytes.
#define QN_STATIC_SCRATCH_DOUBLES (QN_STATIC_MAX_CTAS * (QN_STATIC_MAX_M * (QN_STATIC_MAX_M + 1) / 2 + QN_STATIC_MAX_M))
static __device__ __align__(256) double qn_static_scratch[QN_STATIC_SCRATCH_DOUBLES];

namespace {

constexpr int kMaxDevices = 64;
// Device address of qn_static_scratch per device ordinal.  In host code the array's name is only a
// handle for the runtime, not an address a kernel can use: the address comes from
// cudaGetSymbolAddress, asked once per device with that device current.
double* g_scratch_addr[kMaxDevices];

qn_status scratch_for_current_device(double** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) {
        cudaGetLastError();
        return QN_ERR_CUDA;
    }
    if (!g_scratch_addr[dev]) {
        double* p = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&p), qn_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return QN_ERR_CUDA;
        }
        // Load every kernel this entry point can dispatch to, and raise their shared-memory limits, now: the first
        // use of a kernel loads its code, which may allocate inside the driver, and later calls must not.
        if (qn_solve_init() != cudaSuccess || qn_gram_preload() != cudaSuccess) {
            cudaGetLastError();
            return QN_ERR_CUDA;
        }
        g_scratch_addr[dev] = p;
    }
    *out = g_scratch_addr[dev];
    return QN_OK;
}

}  // namespace

extern "C" qn_status qn_gram_static(int64_t n, int32_t m, qn_dtype dtype, const void* g, double* gram_out,
                                    void* cuda_stream) {
    if (!g || !gram_out || n < 1 || m < 1 || (dtype != QN_F32 && dtype != QN_BF16)) return QN_ERR_INVALID;
    if (m > QN_STATIC_MAX_M) return QN_ERR_INVALID;  // beyond what the static scratch can hold
    double* scratch = nullptr;
    qn_status s = scratch_for_current_device(&scratch);
    if (s != QN_OK) return s;
    cudaStream_t st = static_cast<cudaStream_t>(cuda_stream);
    int np = 0;
    if (qn_launch_gram(dtype, g, n, m, false, scratch, &np, QN_STATIC_MAX_CTAS, st, nullptr) != cudaSuccess)
        return QN_ERR_CUDA;
    qn_solve_params p;
    memset(&p, 0, sizeof(p));
    p.m = m;
    p.source = QN_SRC_PARTIALS;
    p.partials = scratch;
    p.num_partials = np;
    p.gram_out = gram_out;
    p.gram_only = 1;
    p.lambda = 1.0;
    if (qn_launch_solve(p, st, nullptr) != cudaSuccess) return QN_ERR_CUDA;
    return QN_OK;
}
