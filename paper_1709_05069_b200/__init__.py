"""B200 (sm_100a) implementation of the Parameter-Server quasi-Newton step of arXiv 1709.05069.

The work is done by ``libqn.so`` (hand-written CUDA kernels behind a C ABI, declared in
``include/qn.h``); ``paper_1709_05069_b200.qn`` is the thin ctypes binding with the same names.
Importing this package does not load the library; the first call into ``qn`` does, and raises if
the library is missing or no CUDA device is usable -- there is no CPU fallback.
"""
from . import qn  # noqa: F401
from .qn import (  # noqa: F401
    QN_BF16,
    QN_F32,
    QNError,
    Handle,
    qn_create,
    qn_destroy,
    qn_gram,
    qn_push,
    qn_rebuild,
    qn_status_sync,
    qn_strerror,
    qn_update,
    qn_update_host,
    qn_update_window,
)
