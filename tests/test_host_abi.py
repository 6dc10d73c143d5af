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
