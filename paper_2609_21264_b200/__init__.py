"""B200-native fused attention forward pass (sm_100a) behind a small C-ABI library.

`fa_create`, `fa_forward`, `fa_forward_host`, `fa_last_status`, `fa_destroy`
and `fa_strerror` are thin ctypes wrappers of the functions declared in
``include/fa.h``; every step of the computation runs in the CUDA kernels of
``csrc/``.  Importing the package does not load the library; the first call
does, and raises if it is missing (there is no CPU fallback).
"""
from . import metrics, workloads  # noqa: F401

__all__ = ["metrics", "workloads", "binding", "build"]


def __getattr__(name):
    if name in ("binding", "build"):
        import importlib
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
