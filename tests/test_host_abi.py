"""Host-only checks of the C ABI: the library loads without a GPU, exports every symbol that include/qn.h
declares, validates arguments before touching CUDA, and fails loudly (no CPU fallback) without a device."""
import ctypes
import os
import re

import pytest
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def qn():
    from paper_1709_05069_b200 import build as qn_build
    from paper_1709_05069_b200 import qn as mod

    qn_build.build()
    mod.lib()
    return mod


def test_exports_every_declared_symbol(qn):
    header = open(os.path.join(ROOT, "include", "qn.h")).read()
    declared = set(re.findall(r"QN_API\s+[\w\s\*]+?\b(qn_\w+)\s*\(", header))
    assert declared, "no declarations found in include/qn.h"
    L = qn.lib()
    for name in declared:
        assert hasattr(L, name), name
    assert declared == set(qn.EXPORTS)


def test_strerror(qn):
    texts = {qn.qn_strerror(s) for s in range(8)}
    assert len(texts) == 8 and "ok" in texts
    assert qn.qn_strerror(99) == "unknown status"


def test_create_validates_before_cuda(qn):
    L = qn.lib()
    h = ctypes.c_void_p()
    for n, m, dt in ((0, 8, 0), (-5, 8, 0), (100, 0, 0), (100, 65, 0), (100, 8, 2), (100, 8, -1)):
        assert L.qn_create(n, m, dt, ctypes.byref(h)) == qn.QN_ERR_INVALID
    assert L.qn_create(100, 8, 0, None) == qn.QN_ERR_INVALID


def test_null_handle_is_rejected(qn):
    L = qn.lib()
    assert L.qn_destroy(None) == qn.QN_ERR_INVALID
    assert L.qn_update(None, None, None, 1.0, 0.1, None, None, None, None) == qn.QN_ERR_INVALID
    assert L.qn_gram(None, None, None, None) == qn.QN_ERR_INVALID
    assert L.qn_push(None, 0, None, None, None) == qn.QN_ERR_INVALID
    assert L.qn_update_window(None, 1.0, 0.1, None, None, None, None) == qn.QN_ERR_INVALID
    assert L.qn_rebuild(None, None) == qn.QN_ERR_INVALID
    assert L.qn_status_sync(None) == qn.QN_ERR_INVALID
    assert L.qn_last_launches(None) == 0
    assert L.qn_set_sweep_limit(None, 3) == qn.QN_ERR_INVALID
    assert L.qn_set_gram_path(None, 0) == qn.QN_ERR_INVALID


class _FakeCudaTensor:
    """Stands in for a CUDA tensor on a machine without one: the binding's checks read only these attributes."""

    def __init__(self, shape, dtype, index):
        self.shape, self.dtype, self.is_cuda = shape, dtype, True
        self.device = torch.device("cuda", index)

    def is_contiguous(self):
        return True

    def numel(self):
        n = 1
        for s in self.shape:
            n *= s
        return n

    def data_ptr(self):
        raise AssertionError("a tensor on the wrong device must be refused before its pointer is taken")


def test_binding_refuses_tensors_of_another_device(qn):
    """A tensor on another GPU than the handle's would make the kernels dereference memory they cannot reach (a
    device fault, not an error code), so the binding refuses it on the host."""
    h = qn.Handle(0, 100, 4, torch.float32, device=1)
    with pytest.raises(ValueError, match="cuda:0"):
        qn._dev_matrix(_FakeCudaTensor((4, 100), torch.float32, 0), h, "theta")
    with pytest.raises(ValueError, match="cuda:3"):
        qn._dev_vector(_FakeCudaTensor((100,), torch.float32, 3), h, "theta_new")
    with pytest.raises(ValueError, match="cuda:0"):
        qn._check_gram_buffer(h, _FakeCudaTensor((20,), torch.float64, 0))
    with pytest.raises(ValueError, match="same device"):
        g = _FakeCudaTensor((4, 100), torch.float32, 0)
        g.dim = lambda: 2
        qn.qn_gram_static(g, _FakeCudaTensor((20,), torch.float64, 1))
    # the same objects on the handle's device pass the device check and reach data_ptr()
    with pytest.raises(AssertionError):
        qn._dev_matrix(_FakeCudaTensor((4, 100), torch.float32, 1), h, "theta")


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-device behaviour")
def test_no_device_fails_loudly(qn):
    """Without a CUDA device the product path reports an error; it never computes on the CPU."""
    L = qn.lib()
    h = ctypes.c_void_p()
    assert L.qn_create(1000, 8, 0, ctypes.byref(h)) == qn.QN_ERR_CUDA
    assert not h.value
    with pytest.raises(qn.QNError):
        qn.qn_create(1000, 8, torch.float32)


def test_product_does_not_reach_the_oracle():
    """No file of the product package or of the C sources mentions the oracle package."""
    pkg = os.path.join(ROOT, "paper_1709_05069_b200")
    for base, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(base, f)).read()
                assert "oracle" not in text.lower(), os.path.join(base, f)
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_1709_05069_b200" not in text and "libqn.so" not in text and "qn.h" not in text
