"""ctypes binding of libqn.so: the same entry points as ``include/qn.h``, arguments marshalled only.

Tensors are ``torch`` CUDA tensors used purely as device memory (``data_ptr()``); streams are
``torch.cuda`` streams passed by handle.  No arithmetic of the method happens in Python.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

QN_F32 = 0
QN_BF16 = 1
QN_MAX_M = 64
QN_GRAM_PATH_AUTO = 0
QN_GRAM_PATH_PLAIN_ALU = 1
QN_GRAM_PATH_FP64 = 2

(QN_OK, QN_ERR_INVALID, QN_ERR_ALLOC, QN_ERR_CUDA, QN_ERR_STATE, QN_ERR_NOT_CONVERGED, QN_ERR_NONFINITE,
 QN_ERR_DEVICE_TIMEOUT) = range(8)

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libqn.so")
_lib: Optional[ctypes.CDLL] = None

EXPORTS = (
    "qn_strerror", "qn_create", "qn_destroy", "qn_update", "qn_gram", "qn_update_from_gram", "qn_apply_hinv",
    "qn_set_rank_cap", "qn_set_sweep_limit", "qn_set_gram_path", "qn_set_tau_cap", "qn_last_tau", "qn_push",
    "qn_update_window", "qn_rebuild",
    "qn_window_alloc", "qn_window_theta", "qn_window_g", "qn_window_mark_full", "qn_update_host", "qn_status_sync",
    "qn_last_launches", "qn_total_launches", "qn_last_sweeps", "qn_last_gram_kernel", "qn_precision_flag",
    "qn_timing_begin",
    "qn_timing_end",
    "qn_gram_static", "qn_selftest_bounded_wait",
)
TIME_KINDS = ("gram", "solve", "combine", "row")
KERNEL_NAMES = {
    0: "none",
    1: "direct (m <= 8, register-fed, plain ALUs)",
    2: "bulk-copy (m <= 8, shared-memory stages, packed fp32 ALUs, fp64 flush)",
    3: "tiled (plain ALUs)",
    4: "tcgen05 (bf16 hi/lo split, fp32 accumulation in short chains, fp64 flush)",
    5: "row refresh, register-fed",
    6: "row refresh, bulk-copy (fp32 sums per work item, fp64 across)",
}


class QNError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__("%s: %s (status %d)" % (where, qn_strerror(status), status))


def lib() -> ctypes.CDLL:
    """Load libqn.so (built by ``paper_1709_05069_b200.build``).  Raises if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise FileNotFoundError(
                "%s not found: build it with `python -m paper_1709_05069_b200.build` (there is no CPU fallback)" % _LIB_PATH)
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, dbl = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_double
        L.qn_strerror.argtypes, L.qn_strerror.restype = [i32], ctypes.c_char_p
        L.qn_create.argtypes, L.qn_create.restype = [i64, i32, i32, ctypes.POINTER(vp)], i32
        L.qn_destroy.argtypes, L.qn_destroy.restype = [vp], i32
        L.qn_update.argtypes, L.qn_update.restype = [vp, vp, vp, dbl, dbl, vp, vp, vp, vp], i32
        L.qn_gram.argtypes, L.qn_gram.restype = [vp, vp, vp, vp], i32
        L.qn_selftest_bounded_wait.argtypes, L.qn_selftest_bounded_wait.restype = [vp, vp], i32
        L.qn_set_tau_cap.argtypes, L.qn_set_tau_cap.restype = [vp, i32], i32
        L.qn_last_tau.argtypes, L.qn_last_tau.restype = [vp], dbl
        L.qn_set_rank_cap.argtypes, L.qn_set_rank_cap.restype = [vp, i32], i32
        L.qn_set_sweep_limit.argtypes, L.qn_set_sweep_limit.restype = [vp, i32], i32
        L.qn_set_gram_path.argtypes, L.qn_set_gram_path.restype = [vp, i32], i32
        L.qn_apply_hinv.argtypes, L.qn_apply_hinv.restype = [vp, vp, vp, dbl, vp, vp, vp, vp, vp], i32
        L.qn_update_from_gram.argtypes, L.qn_update_from_gram.restype = [vp, vp, vp, vp, dbl, dbl, vp, vp, vp, vp], i32
        L.qn_push.argtypes, L.qn_push.restype = [vp, i32, vp, vp, vp], i32
        L.qn_update_window.argtypes, L.qn_update_window.restype = [vp, dbl, dbl, vp, vp, vp, vp], i32
        L.qn_rebuild.argtypes, L.qn_rebuild.restype = [vp, vp], i32
        L.qn_window_alloc.argtypes, L.qn_window_alloc.restype = [vp], i32
        L.qn_window_theta.argtypes, L.qn_window_theta.restype = [vp], vp
        L.qn_window_g.argtypes, L.qn_window_g.restype = [vp], vp
        L.qn_window_mark_full.argtypes, L.qn_window_mark_full.restype = [vp], i32
        L.qn_update_host.argtypes, L.qn_update_host.restype = [vp, vp, vp, dbl, dbl, vp, vp, vp, vp], i32
        L.qn_status_sync.argtypes, L.qn_status_sync.restype = [vp], i32
        L.qn_last_launches.argtypes, L.qn_last_launches.restype = [vp], i32
        L.qn_total_launches.argtypes, L.qn_total_launches.restype = [vp], i64
        L.qn_last_sweeps.argtypes, L.qn_last_sweeps.restype = [vp], i32
        L.qn_last_gram_kernel.argtypes, L.qn_last_gram_kernel.restype = [vp], i32
        L.qn_precision_flag.argtypes, L.qn_precision_flag.restype = [vp], i32
        L.qn_gram_static.argtypes, L.qn_gram_static.restype = [i64, i32, i32, vp, vp, vp], i32
        L.qn_timing_begin.argtypes, L.qn_timing_begin.restype = [vp, i32], i32
        L.qn_timing_end.argtypes, L.qn_timing_end.restype = [vp, vp, vp], i32
        _lib = L
    return _lib


def qn_strerror(status: int) -> str:
    return lib().qn_strerror(int(status)).decode()


def _check(status: int, where: str, allow=()) -> int:
    if status != QN_OK and status not in allow:
        raise QNError(status, where)
    return status


def dtype_code(dtype: torch.dtype) -> int:
    if dtype == torch.float32:
        return QN_F32
    if dtype == torch.bfloat16:
        return QN_BF16
    raise TypeError("storage dtype must be torch.float32 or torch.bfloat16")


class Handle:
    """Owner of a ``qn_handle``.  ``n``, ``m``, ``dtype`` as passed to ``qn_create``; ``device`` is the index of
    the CUDA device the handle lives on (every tensor passed with it must live there too)."""

    def __init__(self, ptr: int, n: int, m: int, dtype: torch.dtype, device: int = 0):
        self.ptr, self.n, self.m, self.dtype, self.device = ptr, n, m, dtype, device
        self.gram_path = QN_GRAM_PATH_AUTO  # as last set through qn_set_gram_path

    def close(self):
        if self.ptr:
            lib().qn_destroy(self.ptr)
            self.ptr = 0

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()

    @property
    def last_launches(self) -> int:
        return lib().qn_last_launches(self.ptr)

    @property
    def total_launches(self) -> int:
        return lib().qn_total_launches(self.ptr)

    @property
    def last_sweeps(self) -> int:
        return lib().qn_last_sweeps(self.ptr)

    @property
    def last_gram_kernel(self) -> str:
        """Name of the kernel the most recent Gram pass (or row refresh) was dispatched to."""
        code = lib().qn_last_gram_kernel(self.ptr)
        name = KERNEL_NAMES.get(code & 0xff, "unknown")
        return name + (", fp64 products and sums" if code & 0x100 else "")


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _same_device(t, h: Handle, name: str) -> None:
    # a tensor on another GPU would make the kernels dereference memory they cannot reach
    if t.device.index != h.device:
        raise ValueError("%s lives on cuda:%s but the handle was created on cuda:%d" % (name, t.device.index, h.device))


def _dev_matrix(t: torch.Tensor, h: Handle, name: str) -> int:
    if not t.is_cuda or t.dtype != h.dtype or tuple(t.shape) != (h.m, h.n) or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA tensor [m][n] of the handle's dtype" % name)
    _same_device(t, h, name)
    return t.data_ptr()


def _dev_vector(t: torch.Tensor, h: Handle, name: str) -> int:
    if not t.is_cuda or t.dtype != h.dtype or tuple(t.shape) != (h.n,) or not t.is_contiguous():
        raise ValueError("%s must be a contiguous CUDA tensor [n] of the handle's dtype" % name)
    _same_device(t, h, name)
    return t.data_ptr()


def qn_create(n: int, m: int, dtype: torch.dtype) -> Handle:
    """Handle on the current CUDA device (``torch.cuda.current_device()``)."""
    out = ctypes.c_void_p(0)
    device = 0
    if torch.cuda.is_available():
        device = torch.cuda.current_device()
        torch.cuda.set_device(device)  # make torch's device the runtime's current one
    _check(lib().qn_create(int(n), int(m), dtype_code(dtype), ctypes.byref(out)), "qn_create")
    return Handle(out.value, int(n), int(m), dtype, device)


def qn_destroy(h: Handle) -> None:
    h.close()


def _host_outputs(h: Handle, want: bool):
    if not want:
        return None, None, None, None
    j = ctypes.c_int32(0)
    sigma = (ctypes.c_double * h.m)()
    return j, sigma, ctypes.byref(j), ctypes.cast(sigma, ctypes.c_void_p)


def qn_update(h: Handle, theta: torch.Tensor, g: torch.Tensor, tau: float, lam: float, theta_new: torch.Tensor,
              want_host: bool = True, stream=None, allow=(QN_ERR_NOT_CONVERGED, QN_ERR_NONFINITE)):
    """One Server step on device tensors.  Returns (j, sigma list, status) or None when ``want_host`` is False
    (then nothing waits for the device)."""
    j, sigma, jp, sp = _host_outputs(h, want_host)
    st = lib().qn_update(h.ptr, _dev_matrix(theta, h, "theta"), _dev_matrix(g, h, "g"), float(tau), float(lam),
                         _dev_vector(theta_new, h, "theta_new"), jp, sp, _stream_ptr(stream))
    _check(st, "qn_update", allow)
    if want_host:
        return j.value, list(sigma), st
    return None


def qn_gram(h: Handle, g: torch.Tensor, gram_out: torch.Tensor, stream=None) -> None:
    """Centred Gram (m*m) followed by w = G^T gbar (m) into ``gram_out`` (CUDA float64, m*m + m)."""
    _check_gram_buffer(h, gram_out)
    _check(lib().qn_gram(h.ptr, _dev_matrix(g, h, "g"), gram_out.data_ptr(), _stream_ptr(stream)), "qn_gram")


def qn_set_rank_cap(h: Handle, j_cap: Optional[int]) -> None:
    """Keep at most ``j_cap`` modes in later steps on this handle (``None`` or a negative value: no cap)."""
    _check(lib().qn_set_rank_cap(h.ptr, -1 if j_cap is None else int(j_cap)), "qn_set_rank_cap")


def qn_set_sweep_limit(h: Handle, max_sweeps: Optional[int]) -> None:
    """Limit the fp64 Jacobi sweeps of later steps on this handle (``None`` or 0: the built-in limit of 30).  A step
    that reaches the limit still writes its outputs and reports QN_ERR_NOT_CONVERGED."""
    _check(lib().qn_set_sweep_limit(h.ptr, 0 if max_sweeps is None else int(max_sweeps)), "qn_set_sweep_limit")


def qn_set_gram_path(h: Handle, path: int) -> None:
    """``QN_GRAM_PATH_AUTO`` (default), ``QN_GRAM_PATH_PLAIN_ALU`` (register-fed plain-ALU Gram kernels only) or
    ``QN_GRAM_PATH_FP64`` (those kernels with fp64 products and sums whatever n)."""
    _check(lib().qn_set_gram_path(h.ptr, int(path)), "qn_set_gram_path")
    h.gram_path = int(path)


def qn_set_tau_cap(h: Handle, on: bool) -> None:
    """Bound tau by the reciprocal of the method's estimate of the Hessian's largest singular value in later
    ``qn_update`` / ``qn_update_host`` calls on this handle (one more pass, over theta)."""
    _check(lib().qn_set_tau_cap(h.ptr, 1 if on else 0), "qn_set_tau_cap")


def qn_last_tau(h: Handle) -> float:
    """Learning rate used by the most recent step whose results were fetched to the host."""
    return float(lib().qn_last_tau(h.ptr))


def qn_apply_hinv(h: Handle, theta: torch.Tensor, g: torch.Tensor, lam: float, z: torch.Tensor, out: torch.Tensor,
                  want_host: bool = True, stream=None, allow=(QN_ERR_NOT_CONVERGED, QN_ERR_NONFINITE)):
    """``out = Hbar^{-1} z`` (Eq. (3)/(4)) for an arbitrary device vector ``z``.  Returns like ``qn_update``."""
    j, sigma, jp, sp = _host_outputs(h, want_host)
    st = lib().qn_apply_hinv(h.ptr, _dev_matrix(theta, h, "theta"), _dev_matrix(g, h, "g"), float(lam),
                             _dev_vector(z, h, "z"), _dev_vector(out, h, "out"), jp, sp, _stream_ptr(stream))
    _check(st, "qn_apply_hinv", allow)
    if want_host:
        return j.value, list(sigma), st
    return None


def _check_gram_buffer(h: Handle, gram: torch.Tensor) -> None:
    if not gram.is_cuda or gram.dtype != torch.float64 or gram.numel() != h.m * h.m + h.m or not gram.is_contiguous():
        raise ValueError("the Gram buffer must be a contiguous CUDA float64 tensor with m*m + m elements")
    _same_device(gram, h, "the Gram buffer")


def qn_update_from_gram(h: Handle, theta: torch.Tensor, g: torch.Tensor, gram: torch.Tensor, tau: float, lam: float,
                        theta_new: torch.Tensor, want_host: bool = True, stream=None,
                        allow=(QN_ERR_NOT_CONVERGED, QN_ERR_NONFINITE)):
    """The step without its Gram pass: ``gram`` is what ``qn_gram`` wrote, or the sum of such buffers over the
    column slices of an n-sharded problem.  Returns like ``qn_update``."""
    _check_gram_buffer(h, gram)
    j, sigma, jp, sp = _host_outputs(h, want_host)
    st = lib().qn_update_from_gram(h.ptr, _dev_matrix(theta, h, "theta"), _dev_matrix(g, h, "g"), gram.data_ptr(),
                                   float(tau), float(lam), _dev_vector(theta_new, h, "theta_new"), jp, sp,
                                   _stream_ptr(stream))
    _check(st, "qn_update_from_gram", allow)
    if want_host:
        return j.value, list(sigma), st
    return None


def shard_columns(n: int, world: int, rank: int, align: int = 8):
    """Column range [begin, end) of ``rank`` when n columns are split over ``world`` ranks in contiguous slices whose
    boundaries are multiples of ``align`` (so that every slice keeps 16-byte aligned rows).  Host logic only."""
    if world < 1 or not 0 <= rank < world or n < 0 or align < 1:
        raise ValueError("bad shard request")
    blocks = (n + align - 1) // align
    b0 = blocks * rank // world
    b1 = blocks * (rank + 1) // world
    return min(b0 * align, n), min(b1 * align, n)


def qn_update_sharded(h: Handle, theta: torch.Tensor, g: torch.Tensor, tau: float, lam: float, theta_new: torch.Tensor,
                      gram_buf: torch.Tensor, group=None, want_host: bool = True, stream=None):
    """One Server step on this rank's column slice of an n-sharded problem (one process per GPU).

    ``theta``, ``g``: [m][n_local] of this rank; ``gram_buf``: CUDA float64 scratch with m*m + m elements.  The only
    exchange is one all-reduce of ``gram_buf`` (``torch.distributed``, NCCL between GPUs); every other byte stays on
    its GPU.  With no initialised process group this is ``qn_gram`` + ``qn_update_from_gram``; with a group of one
    rank the all-reduce still runs (it is the identity).

    The collective is ordered against torch's CURRENT stream, so the three calls run with ``stream`` made current:
    the all-reduce then sits between the Gram pass and the step on the same stream.

    With ``want_host`` the step's precision flag is read as well (``qn_precision_flag``): if the spectrum has a
    retained mode too small for the reduced-precision Gram pass, the three calls are repeated once with the handle on
    ``QN_GRAM_PATH_FP64``.  sigma and j are identical on every rank, so all ranks repeat together.  Without
    ``want_host`` nothing is read back and nothing is repeated."""
    import torch.distributed as dist

    if stream is None:
        stream = torch.cuda.current_stream()

    def three_calls():
        qn_gram(h, g, gram_buf, stream=stream)
        if dist.is_available() and dist.is_initialized():
            dist.all_reduce(gram_buf, op=dist.ReduceOp.SUM, group=group)
        return qn_update_from_gram(h, theta, g, gram_buf, tau, lam, theta_new, want_host=want_host, stream=stream)

    with torch.cuda.stream(stream):
        res = three_calls()
        if want_host and lib().qn_precision_flag(h.ptr):
            before = h.gram_path
            qn_set_gram_path(h, QN_GRAM_PATH_FP64)
            try:
                res = three_calls()
            finally:
                qn_set_gram_path(h, before)
        return res


def qn_push(h: Handle, slot: int, theta_col: torch.Tensor, g_col: torch.Tensor, stream=None) -> None:
    _check(lib().qn_push(h.ptr, int(slot), _dev_vector(theta_col, h, "theta_col"), _dev_vector(g_col, h, "g_col"),
                         _stream_ptr(stream)), "qn_push")


def qn_update_window(h: Handle, tau: float, lam: float, theta_new: torch.Tensor, want_host: bool = True, stream=None,
                     allow=(QN_ERR_NOT_CONVERGED, QN_ERR_NONFINITE)):
    j, sigma, jp, sp = _host_outputs(h, want_host)
    st = lib().qn_update_window(h.ptr, float(tau), float(lam), _dev_vector(theta_new, h, "theta_new"), jp, sp,
                                _stream_ptr(stream))
    _check(st, "qn_update_window", allow)
    if want_host:
        return j.value, list(sigma), st
    return None


def qn_rebuild(h: Handle, stream=None) -> None:
    _check(lib().qn_rebuild(h.ptr, _stream_ptr(stream)), "qn_rebuild")


def qn_window_alloc(h: Handle) -> None:
    _check(lib().qn_window_alloc(h.ptr), "qn_window_alloc")


def qn_window_ptrs(h: Handle) -> Tuple[int, int]:
    return lib().qn_window_theta(h.ptr) or 0, lib().qn_window_g(h.ptr) or 0


def qn_window_mark_full(h: Handle) -> None:
    _check(lib().qn_window_mark_full(h.ptr), "qn_window_mark_full")


def qn_update_host(h: Handle, theta_host: torch.Tensor, g_host: torch.Tensor, tau: float, lam: float,
                   theta_new_host: torch.Tensor, stream=None, allow=(QN_ERR_NOT_CONVERGED, QN_ERR_NONFINITE)):
    """The step with HOST tensors (pinned recommended): copies in, computes, copies theta_new out, waits."""
    for t, shape, name in ((theta_host, (h.m, h.n), "theta_host"), (g_host, (h.m, h.n), "g_host"),
                           (theta_new_host, (h.n,), "theta_new_host")):
        if t.is_cuda or t.dtype != h.dtype or tuple(t.shape) != shape or not t.is_contiguous():
            raise ValueError("%s must be a contiguous host tensor of shape %s and the handle's dtype" % (name, shape))
    j, sigma, jp, sp = _host_outputs(h, True)
    st = lib().qn_update_host(h.ptr, theta_host.data_ptr(), g_host.data_ptr(), float(tau), float(lam),
                              theta_new_host.data_ptr(), jp, sp, _stream_ptr(stream))
    _check(st, "qn_update_host", allow)
    return j.value, list(sigma), st


def qn_selftest_bounded_wait(h: Handle, stream=None) -> None:
    """Enqueue the bounded-wait self-test: the next step on ``h`` reports QN_ERR_DEVICE_TIMEOUT."""
    _check(lib().qn_selftest_bounded_wait(h.ptr, _stream_ptr(stream)), "qn_selftest_bounded_wait")


def qn_status_sync(h: Handle) -> int:
    return lib().qn_status_sync(h.ptr)


def qn_timing_begin(h: Handle, max_kernels: int) -> None:
    _check(lib().qn_timing_begin(h.ptr, int(max_kernels)), "qn_timing_begin")


def qn_timing_end(h: Handle):
    """{kind: (total_ms, launches)} for the kernels launched since ``qn_timing_begin``."""
    ms = (ctypes.c_double * len(TIME_KINDS))()
    cnt = (ctypes.c_int32 * len(TIME_KINDS))()
    _check(lib().qn_timing_end(h.ptr, ctypes.cast(ms, ctypes.c_void_p), ctypes.cast(cnt, ctypes.c_void_p)),
           "qn_timing_end")
    return {k: (ms[i], cnt[i]) for i, k in enumerate(TIME_KINDS)}


QN_STATIC_MAX_M = 32


def qn_gram_static(g: torch.Tensor, gram_out: torch.Tensor, stream=None) -> None:
    """``qn_gram`` for callers that must not allocate: no handle, scratch in a fixed array inside the library.

    ``g`` is a contiguous CUDA tensor [m][n] (float32 or bfloat16, m <= 32), ``gram_out`` a CUDA float64
    tensor with m*m + m elements.  Calls on one device share the scratch: do not let two overlap."""
    if not g.is_cuda or g.dim() != 2 or not g.is_contiguous():
        raise ValueError("g must be a contiguous CUDA tensor [m][n]")
    m, n = g.shape
    if not gram_out.is_cuda or gram_out.dtype != torch.float64 or gram_out.numel() != m * m + m \
            or not gram_out.is_contiguous():
        raise ValueError("gram_out must be a contiguous CUDA float64 tensor with m*m + m elements")
    if gram_out.device != g.device:
        raise ValueError("g and gram_out must live on the same device")
    # the call runs on the runtime's current device: make that the tensors' device for its duration
    with torch.cuda.device(g.device):
        _check(lib().qn_gram_static(int(n), int(m), dtype_code(g.dtype), g.data_ptr(), gram_out.data_ptr(),
                                    _stream_ptr(stream)), "qn_gram_static")
