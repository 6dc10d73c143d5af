"""The allocation-free Gram entry point, qn_gram_static, against the handle-based qn_gram and the CPU oracle.

Collected last on purpose (file name): a run that stops at the first failure has then already run
every other test.  The entry point serves callers that cannot allocate device memory while running
(inside a framework whose allocator owns the GPU's memory, or under a no-cudaMalloc-after-start-up
rule), so the test also checks that calling it leaves the CUDA context's allocated memory unchanged.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("dtype,m,n", [("f32", 8, 300_001), ("bf16", 16, 200_000), ("f32", 32, 5_000_000)])
def test_static_gram_matches_handle_gram_twice(dtype, m, n):
    from paper_1709_05069_b200 import qn

    assert torch.cuda.is_available()
    outs_static, outs_handle = [], []
    # two calls in a row on different inputs: the second must not be affected by what the first left
    # in the shared scratch array
    for call in range(2):
        cfg = W.Config(20 + call, n, m, dtype, -1, 1, 0, 0.05, 1e-3, 0.5, 0.05)
        _, g = W.generate(cfg, "cuda")
        a = torch.full((m * m + m,), float("nan"), dtype=torch.float64, device="cuda")
        b = torch.full((m * m + m,), float("nan"), dtype=torch.float64, device="cuda")
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        qn.qn_gram_static(g, a)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        if call == 1:  # the first call on a device may load the module that holds the array
            assert free_after == free_before
        with qn.qn_create(n, m, g.dtype) as h:
            qn.qn_gram(h, g, b)
            torch.cuda.synchronize()
        outs_static.append(a.cpu().numpy())
        outs_handle.append(b.cpu().numpy())
        # and against the definition: the oracle's centred Gram and a plain product for G^T gbar
        C = outs_static[-1][: m * m].reshape(m, m)
        w = outs_static[-1][m * m:]
        Cref = oracle.gram(W.to_bits(g))
        # below 2^17 columns (2^22 for m <= 8) every product and sum is fp64; above, with m > 8, the tensor cores add in fp32 and
        # truncate, which scales the whole Gram down by a few 1e-7 (harmless for sigma_k / sigma_1 and the update)
        assert np.max(np.abs(C - Cref)) <= (2e-9 if (n < (1 << 17) or m <= 8) else 1e-6) * np.abs(Cref).max()
        assert np.array_equal(C, C.T)
        g64 = oracle.storage_to_f64(W.to_bits(g))
        gbar = g64.mean(0)
        wref = (g64 - gbar) @ gbar
        assert np.max(np.abs(w - wref)) <= 1e-7 * np.linalg.norm(g64 - gbar, axis=1).max() * np.linalg.norm(gbar)
    for a, b in zip(outs_static, outs_handle):
        assert np.all(np.isfinite(a))
        scale = np.abs(b[: m * m]).max()
        assert np.max(np.abs(a[: m * m] - b[: m * m])) <= 2e-9 * scale  # the Gram tolerance of test_gram_entry_point
        wscale = max(np.abs(b[m * m:]).max(), 1e-300)
        assert np.max(np.abs(a[m * m:] - b[m * m:])) <= 1e-7 * wscale
    assert not np.array_equal(outs_static[0], outs_static[1])


def test_static_gram_allocates_nothing_for_a_new_shape_class_after_warm_up():
    """The first call on a device loads every kernel variant the entry point can dispatch to; a later call of
    another dtype, Worker count, size class or alignment must leave the device's free memory unchanged."""
    from paper_1709_05069_b200 import qn

    warm = torch.randn(4, 1000, device="cuda")
    qn.qn_gram_static(warm, torch.empty(4 * 4 + 4, dtype=torch.float64, device="cuda"))
    torch.cuda.synchronize()
    shapes = [("bf16", 8, (1 << 22) + 8), ("f32", 24, 1 << 22), ("bf16", 12, 40_000), ("f32", 3, 12_345),
              ("bf16", 32, (1 << 22) + 64), ("f32", 6, 1 << 22)]
    inputs = []
    for i, (dtype, m, n) in enumerate(shapes):
        cfg = W.Config(30 + i, n, m, dtype, -1, 1, 0, 0.05, 1e-3, 0.5, 0.05)
        _, g = W.generate(cfg, "cuda")
        inputs.append((g, torch.full((m * m + m,), float("nan"), dtype=torch.float64, device="cuda")))
    unaligned = torch.randn(5 * 3001 + 1, device="cuda")[1:].view(5, 3001)  # rows off the 16-byte boundaries
    inputs.append((unaligned, torch.empty(5 * 5 + 5, dtype=torch.float64, device="cuda")))
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for g, out in inputs:
        qn.qn_gram_static(g, out)
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    for g, out in inputs:
        assert bool(torch.isfinite(out).all())


def test_static_gram_rejects_sizes_beyond_its_scratch():
    from paper_1709_05069_b200 import qn

    L = qn.lib()
    g = torch.zeros(33, 64, device="cuda")
    out = torch.zeros(33 * 33 + 33, dtype=torch.float64, device="cuda")
    st = torch.cuda.current_stream().cuda_stream
    assert L.qn_gram_static(64, 33, 0, g.data_ptr(), out.data_ptr(), st) == qn.QN_ERR_INVALID
    assert L.qn_gram_static(0, 8, 0, g.data_ptr(), out.data_ptr(), st) == qn.QN_ERR_INVALID
    assert L.qn_gram_static(64, 8, 0, None, out.data_ptr(), st) == qn.QN_ERR_INVALID
    assert L.qn_gram_static(64, 8, 5, g.data_ptr(), out.data_ptr(), st) == qn.QN_ERR_INVALID
    with pytest.raises(qn.QNError):
        qn.qn_gram_static(g, out)
