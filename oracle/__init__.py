"""ctypes front end of the fp64 CPU oracle (``qn_oracle.c``).

TEST INFRASTRUCTURE ONLY.  The oracle is the checker for the CUDA library and the CPU baseline the
benchmark times.  Only the tests, the smoke check and the benchmark's CPU-baseline / reference legs
may import this package; the product package never does, and this package never imports it.

Arrays are numpy: ``theta`` and ``g`` are C-contiguous ``[m][n]`` (row k = Worker k) of dtype
``float32`` or, for bf16 storage, ``uint16`` holding the bf16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_DIR = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_DIR, "qn_oracle.c")
_LIB = os.path.join(_DIR, "libqn_oracle.so")

F32 = 0
BF16 = 1

_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile ``qn_oracle.c`` with gcc (-O2, no fast-math, OpenMP) if the library is stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fPIC", "-shared", "-fopenmp", "-Wall", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        i64, i32, dbl, vp = ctypes.c_int64, ctypes.c_int, ctypes.c_double, ctypes.c_void_p
        L.qno_gram.argtypes = [i64, i32, i32, vp, vp, i32]
        L.qno_eig.argtypes = [i32, vp, vp, vp]
        L.qno_cutoff.argtypes = [i32, vp, dbl, vp]
        L.qno_update.argtypes = [i64, i32, i32, vp, vp, dbl, dbl, vp, vp, i64, vp, vp, vp, vp, i32]
        L.qno_update_capped.argtypes = [i64, i32, i32, vp, vp, dbl, dbl, i32, i32, vp, vp, i64, vp, vp, vp, vp, vp, i32]
        L.qno_apply_hinv.argtypes = [i64, i32, i32, vp, vp, dbl, vp, vp, vp, i32]
        L.qno_left_vectors.argtypes = [i64, i32, i32, vp, vp, dbl, vp, vp, vp, vp]
        L.qno_round_storage.argtypes = [i64, i32, vp, vp]
        L.qno_round_storage.restype = None
        L.qno_threads_used.argtypes = [i32]
        for f in ("qno_gram", "qno_eig", "qno_cutoff", "qno_update", "qno_update_capped", "qno_apply_hinv",
                  "qno_left_vectors", "qno_threads_used"):
            getattr(L, f).restype = i32
        _lib = L
    return _lib


def _dtype_code(a: np.ndarray) -> int:
    if a.dtype == np.float32:
        return F32
    if a.dtype == np.uint16:
        return BF16
    raise TypeError("storage arrays must be float32 or uint16 (bf16 bits), got %s" % a.dtype)


def _check_pair(theta: Optional[np.ndarray], g: np.ndarray):
    if g.ndim != 2 or not g.flags.c_contiguous:
        raise ValueError("g must be a C-contiguous [m][n] array")
    if theta is not None and (theta.shape != g.shape or theta.dtype != g.dtype or not theta.flags.c_contiguous):
        raise ValueError("theta must match g in shape, dtype and layout")
    return g.shape[0], g.shape[1], _dtype_code(g)


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _raise(rc: int, what: str):
    if rc:
        raise RuntimeError("%s failed: %s" % (what, {1: "bad argument", 2: "out of memory",
                                                     3: "Jacobi did not converge"}.get(rc, rc)))


def threads_used(nthreads: int = 0) -> int:
    return lib().qno_threads_used(nthreads)


def gram(g: np.ndarray, nthreads: int = 0) -> np.ndarray:
    """Centred Gram G^T G (m x m) of the gradient columns (Section 2)."""
    m, n, dt = _check_pair(None, g)
    C = np.empty((m, m), dtype=np.float64)
    _raise(lib().qno_gram(n, m, dt, _ptr(g), _ptr(C), nthreads), "qno_gram")
    return C


def eig(C: np.ndarray):
    """Eigenpairs of a symmetric matrix by cyclic Jacobi: (mu descending, V with v_k in column k)."""
    C = np.ascontiguousarray(C, dtype=np.float64)
    m = C.shape[0]
    V = np.empty((m, m), dtype=np.float64)
    mu = np.empty(m, dtype=np.float64)
    _raise(lib().qno_eig(m, _ptr(C), _ptr(V), _ptr(mu)), "qno_eig")
    return mu, V


def cutoff(mu: np.ndarray, lam: float):
    """(sigma, j) from eigenvalues by the lambda rule of Section 2."""
    mu = np.ascontiguousarray(mu, dtype=np.float64)
    sigma = np.empty_like(mu)
    j = lib().qno_cutoff(len(mu), _ptr(mu), float(lam), _ptr(sigma))
    return sigma, j


class UpdateResult:
    __slots__ = ("theta_new", "j", "sigma", "V", "alpha", "tau_eff")

    def __init__(self, theta_new, j, sigma, V, alpha, tau_eff=None):
        self.theta_new, self.j, self.sigma, self.V, self.alpha, self.tau_eff = theta_new, j, sigma, V, alpha, tau_eff


def update(theta: np.ndarray, g: np.ndarray, tau: float, lam: float, sample_idx: Optional[np.ndarray] = None,
           nthreads: int = 0, want_theta: bool = True, j_cap: Optional[int] = None,
           tau_cap: bool = False) -> UpdateResult:
    """Eq. (2): theta_new = thetabar - tau * Hinv gbar, in fp64.

    With ``sample_idx`` (int64 column indices) only those entries of theta_new are evaluated.  ``j_cap`` keeps at
    most that many of the modes that the lambda rule retains (the largest ones).  ``tau_cap`` bounds tau by
    1 / max_k (sigma_k / ||Theta v_k||), the method's own estimate of the Hessian's largest singular value
    (Section 3, last paragraph); the rate used is returned as ``tau_eff``."""
    m, n, dt = _check_pair(theta, g)
    idx = None
    cnt = n
    if sample_idx is not None:
        idx = np.ascontiguousarray(sample_idx, dtype=np.int64)
        cnt = len(idx)
    out = np.empty(cnt, dtype=np.float64) if want_theta else None
    sigma = np.empty(m, dtype=np.float64)
    V = np.empty((m, m), dtype=np.float64)
    alpha = np.empty(m, dtype=np.float64)
    j = ctypes.c_int(0)
    tau_eff = ctypes.c_double(0.0)
    rc = lib().qno_update_capped(n, m, dt, _ptr(theta), _ptr(g), float(tau), float(lam),
                                 -1 if j_cap is None else int(j_cap), 1 if tau_cap else 0, _ptr(out), _ptr(idx), cnt,
                                 ctypes.byref(j), _ptr(sigma), _ptr(V), _ptr(alpha), ctypes.byref(tau_eff), nthreads)
    _raise(rc, "qno_update")
    return UpdateResult(out, j.value, sigma, V, alpha, tau_eff.value)


def apply_hinv(theta: np.ndarray, g: np.ndarray, lam: float, z: np.ndarray, nthreads: int = 0):
    """Eq. (3)/(4) applied to an arbitrary vector z (n doubles). Returns (Hinv z, j)."""
    m, n, dt = _check_pair(theta, g)
    z = np.ascontiguousarray(z, dtype=np.float64)
    if z.shape != (n,):
        raise ValueError("z must have n entries")
    out = np.empty(n, dtype=np.float64)
    j = ctypes.c_int(0)
    _raise(lib().qno_apply_hinv(n, m, dt, _ptr(theta), _ptr(g), float(lam), _ptr(z), _ptr(out), ctypes.byref(j),
                                nthreads), "qno_apply_hinv")
    return out, j.value


def left_vectors(theta: np.ndarray, g: np.ndarray, lam: float):
    """(U [n][j], Y [n][j], sigma [m], j): the retained u_k and y_k = Theta v_k, for small n."""
    m, n, dt = _check_pair(theta, g)
    U = np.zeros((n, m), dtype=np.float64)
    Y = np.zeros((n, m), dtype=np.float64)
    sigma = np.empty(m, dtype=np.float64)
    j = ctypes.c_int(0)
    # the C routine packs rows with stride j; call once to learn j, then reshape
    bufU = np.zeros(n * m, dtype=np.float64)
    bufY = np.zeros(n * m, dtype=np.float64)
    _raise(lib().qno_left_vectors(n, m, dt, _ptr(theta), _ptr(g), float(lam), _ptr(bufU), _ptr(bufY), _ptr(sigma),
                                  ctypes.byref(j)), "qno_left_vectors")
    jj = j.value
    U = bufU[: n * jj].reshape(n, jj).copy()
    Y = bufY[: n * jj].reshape(n, jj).copy()
    return U, Y, sigma, jj


def round_storage(x: np.ndarray, like: np.ndarray) -> np.ndarray:
    """Round fp64 values once (nearest-even) to the storage type of ``like``."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    out = np.empty(x.shape, dtype=like.dtype)
    lib().qno_round_storage(x.size, _dtype_code(like), _ptr(x), _ptr(out))
    return out


def storage_to_f64(a: np.ndarray) -> np.ndarray:
    """Exact promotion of storage bits (float32, or uint16 bf16 patterns) to float64."""
    if a.dtype == np.float32:
        return a.astype(np.float64)
    if a.dtype == np.uint16:
        return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    raise TypeError(a.dtype)
