"""Helpers shared by the GPU parity tests: guarded output buffers, the comparison with the fp64 CPU oracle, raw
device copies for the window's storage."""
import numpy as np
import torch

import oracle
import workloads as W

TOL = {"f32": 1e-5, "bf16": 2e-3}

GUARD = 128  # elements on each side of an output: 256 bytes for bf16, 512 for fp32, 1 KB for fp64


class Guarded:
    """An output buffer of ``n`` elements with GUARD elements of a fixed bit pattern (a NaN) on both sides, standing
    in for a memory checker: ``check()`` fails if a kernel wrote outside the n elements it was given.  The view keeps
    the alignment of a fresh allocation (the guards are multiples of 256 bytes)."""

    def __init__(self, n, dtype, device="cuda"):
        self.n = n
        self.full = torch.full((n + 2 * GUARD,), float("nan"), dtype=dtype, device=device)
        self.view = self.full[GUARD:GUARD + n]
        self.bits = {torch.float32: torch.int32, torch.bfloat16: torch.int16, torch.float64: torch.int64}[dtype]
        self.pattern = self.full[:1].view(self.bits).clone()

    def check(self):
        raw = self.full.view(self.bits)
        assert bool((raw[:GUARD] == self.pattern).all()), "write before the start of an output buffer"
        assert bool((raw[GUARD + self.n:] == self.pattern).all()), "write past the end of an output buffer"


def run_gpu(qn, theta, g, tau, lam):
    m, n = theta.shape
    guarded = Guarded(n, theta.dtype)
    out = guarded.view
    with qn.qn_create(n, m, theta.dtype) as h:
        j, sigma, status = qn.qn_update(h, theta, g, tau, lam, out)
        launches = h.last_launches
        run_gpu.last_kernel = h.last_gram_kernel  # which Gram kernel delivered the result
    guarded.check()
    return out, j, np.array(sigma), status, launches


def step_launches(n, base=3, m=64):
    """Kernels of one step: from 2^22 parameters on (2^17 with more than 8 Workers: tensor cores) the Gram pass has
    reduced precision, and unless lambda is so large that no retained mode can need it, the step enqueues a
    conditional fp64 repeat of the pass and of the solve (both return at once unless the spectrum asks for them)."""
    return (base,) if n < ((1 << 17) if m > 8 else (1 << 22)) else (base, base + 2)


def _cudart():
    import ctypes

    rt = ctypes.CDLL("libcudart.so.12")  # the runtime torch has loaded
    rt.cudaMemcpy.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_int]
    rt.cudaMemcpy.restype = ctypes.c_int
    return rt


def copy_device_bytes(dst_ptr, src_ptr, nbytes):
    """Device-to-device copy between raw pointers (the window's storage is only known by its address)."""
    torch.cuda.synchronize()
    assert _cudart().cudaMemcpy(dst_ptr, src_ptr, nbytes, 3) == 0
    torch.cuda.synchronize()


def window_bits(qn, h, dtype):
    """The window's (theta, g) storage as numpy bit arrays [m][n]."""
    pt, pg = qn.qn_window_ptrs(h)
    assert pt and pg
    res = []
    for ptr in (pt, pg):
        t = torch.empty((h.m, h.n), dtype=dtype, device="cuda")
        copy_device_bytes(t.data_ptr(), ptr, t.numel() * t.element_size())
        res.append(W.to_bits(t))
    return res


def check_against_oracle(qn, theta, g, tau, lam, dtype, expect_j=None, sample=None):
    out, j, sigma, status, launches = run_gpu(qn, theta, g, tau, lam)
    tb, gb = W.to_bits(theta), W.to_bits(g)
    ref = oracle.update(tb, gb, tau, lam, sample_idx=sample)
    assert status == 0
    assert launches in step_launches(theta.shape[1], 3, theta.shape[0])
    assert j == ref.j, (j, ref.j, sigma / sigma[0], ref.sigma / ref.sigma[0])
    if expect_j is not None:
        assert j == expect_j
    s1 = ref.sigma[0]
    assert np.max(np.abs(sigma - ref.sigma)) <= 1e-5 * s1
    if j:
        assert np.max(np.abs(sigma[:j] - ref.sigma[:j]) / ref.sigma[:j]) <= 1e-5
    got = oracle.storage_to_f64(W.to_bits(out))
    if sample is not None:
        got = got[sample]
    rel = np.linalg.norm(got - ref.theta_new) / np.linalg.norm(ref.theta_new)
    if len(got) < 64:
        # With a handful of elements the L2 figure is not an average.  Bound every element instead: the
        # fp32 combination is accurate to 1e-5 of the magnitude of the terms it adds (thetabar, tau*z_perp
        # and tau*sum alpha_k y_k / sigma_k, which may cancel), and for bf16 storage the single output
        # rounding adds at most one bf16 ulp (2^-8 relative, 2^-133 absolute).
        t64, g64 = oracle.storage_to_f64(tb), oracle.storage_to_f64(gb)
        U, Y, sg, jj = oracle.left_vectors(tb, gb, lam)
        al = ref.alpha[:jj]
        scale = np.abs(t64.mean(0)) + abs(tau) * (np.abs(g64.mean(0)) + np.abs(U) @ np.abs(al)
                                                  + np.abs(Y) @ np.abs(al / sg[:jj]))
        if sample is not None:
            scale = scale[sample]
        bound = 1e-5 * scale
        if dtype == "bf16":
            bound = bound + 2.0 ** -8 * np.abs(ref.theta_new) + 2.0 ** -133
        assert np.all(np.abs(got - ref.theta_new) <= bound), (got, ref.theta_new, bound)
    else:
        assert rel <= TOL[dtype], rel
    return rel, j, out


def assert_gap(theta, g, lam):
    """The generator's promise: a clear gap around lam*sigma_1 in fp64 on the rounded data."""
    ref = oracle.update(W.to_bits(theta), W.to_bits(g), 1.0, lam, want_theta=False)
    j, s = ref.j, ref.sigma
    assert s[j - 1] >= 2 * lam * s[0]
    assert s[j] <= lam * s[0] / 2
    return j
