"""ctypes binding of the C ABI in ``include/fa.h`` -- argument marshalling only.

Function names and argument order follow the header.  Pointers are plain
integers (``tensor.data_ptr()``, ``stream.cuda_stream``); `forward` is a small
convenience that takes torch tensors, allocates O and lse with torch (device
memory plumbing) and calls `fa_forward`.  There is no fallback: if the library
is missing or the call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os

from . import build as _build

FA_OK = 0
FA_ERR_INVALID_ARG = 1
FA_ERR_UNSUPPORTED = 2
FA_ERR_CUDA = 3
FA_ERR_DEVICE_TIMEOUT = 4
FA_ERR_NO_DEVICE = 5
FA_ERR_OOM = 6
FA_FLAG_SERIAL_KERNEL = 1
FA_FLAG_DEBUG_DROP_V_LOAD = 2
FA_FLAG_NO_DEPENDENT_LAUNCH = 4
FA_FLAG_NO_PERSISTENT = 8
FA_FLAG_FORCE_PERSISTENT = 16
FA_FLAG_STREAM_KERNEL = 32
FA_FLAG_NO_STREAM_KERNEL = 64
FA_FLAG_NO_HEAD_PACKING = 128
FA_FLAG_LEGACY_PAIR_KERNEL = 256
FA_FLAG_TWO_CTA_KERNEL = 512
FA_FLAG_QUAD_KERNEL = 1024

EXPORTS = ("fa_create", "fa_forward", "fa_forward_strided", "fa_forward_varlen", "fa_forward_fp8", "fa_forward_mxfp8", "fa_plan", "fa_forward_host", "fa_last_status", "fa_destroy",
           "fa_strerror", "fa_launch_count", "fa_last_kernel_name", "fa_last_kv_splits",
           "fa_forward_split_noalloc", "fa_noalloc_scratch_bytes", "fa_noalloc_last_status", "fa_debug_set_drop_v_load")


class FaError(RuntimeError):
    def __init__(self, status: int, what: str):
        super().__init__("%s: %s (status %d)" % (what, fa_strerror(status), status))
        self.status = status


class fa_config(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("device", ctypes.c_int32),
                ("flags", ctypes.c_uint32), ("wait_limit_ms", ctypes.c_uint32),
                ("kv_splits", ctypes.c_uint32), ("scratch_bytes", ctypes.c_uint64)]


_lib = None


def library_path() -> str:
    return _build.LIB_PATH


class fa_plan_info(ctypes.Structure):
    _fields_ = [("kernel", ctypes.c_char_p), ("kv_splits", ctypes.c_int32), ("ctas", ctypes.c_int64),
                ("heads_per_tile", ctypes.c_int32), ("estimate_pair_us", ctypes.c_double), ("estimate_stream_us", ctypes.c_double)]


def load():
    """Load libfa_b200.so (built in-tree by ``build.build()``); raises if it is missing."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise ImportError("CUDA library %s is missing; run `python -m paper_2609_21264_b200.build` "
                          "(there is no CPU fallback)" % path)
    lib = ctypes.CDLL(path)
    vp, i32, f32 = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    lib.fa_create.restype = i32
    lib.fa_create.argtypes = [ctypes.POINTER(vp), ctypes.POINTER(fa_config)]
    fwd_args = [vp, vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, f32, vp]
    lib.fa_forward.restype = i32
    lib.fa_forward.argtypes = fwd_args
    lib.fa_forward_host.restype = i32
    lib.fa_forward_host.argtypes = fwd_args
    lib.fa_forward_varlen.restype = i32
    lib.fa_forward_varlen.argtypes = [vp] * 8 + [i32] * 8 + [i32, ctypes.c_float, vp]
    lib.fa_plan.restype = i32
    lib.fa_plan.argtypes = [i32, ctypes.POINTER(fa_config), i32] + [i32] * 8 + [ctypes.POINTER(fa_plan_info)]
    lib.fa_forward_fp8.restype = i32
    lib.fa_forward_fp8.argtypes = [vp] * 9 + [i32] * 7 + [f32, vp]
    lib.fa_forward_mxfp8.restype = i32
    lib.fa_forward_mxfp8.argtypes = [vp] * 9 + [i32] * 7 + [f32, vp]
    lib.fa_forward_strided.restype = i32
    lib.fa_forward_strided.argtypes = fwd_args[:-1] + [vp, vp, vp, vp, vp]
    lib.fa_last_status.restype = i32
    lib.fa_last_status.argtypes = [vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.fa_destroy.restype = i32
    lib.fa_destroy.argtypes = [vp]
    lib.fa_strerror.restype = ctypes.c_char_p
    lib.fa_strerror.argtypes = [i32]
    lib.fa_launch_count.restype = ctypes.c_uint64
    lib.fa_launch_count.argtypes = [vp]
    lib.fa_last_kernel_name.restype = ctypes.c_char_p
    lib.fa_last_kernel_name.argtypes = [vp]
    lib.fa_last_kv_splits.restype = i32
    lib.fa_last_kv_splits.argtypes = [vp]
    lib.fa_forward_split_noalloc.restype = i32
    lib.fa_forward_split_noalloc.argtypes = [vp, vp, vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, f32, i32, vp]
    lib.fa_noalloc_scratch_bytes.restype = ctypes.c_size_t
    lib.fa_noalloc_scratch_bytes.argtypes = []
    lib.fa_debug_set_drop_v_load.restype = i32
    lib.fa_debug_set_drop_v_load.argtypes = [vp, i32]
    lib.fa_noalloc_last_status.restype = i32
    lib.fa_noalloc_last_status.argtypes = [ctypes.POINTER(ctypes.c_uint32)]
    _lib = lib
    return lib


def fa_strerror(status: int) -> str:
    return load().fa_strerror(int(status)).decode()


def fa_create(device: int = -1, flags: int = 0, wait_limit_ms: int = 0, kv_splits: int = 0,
              scratch_bytes: int = 0) -> int:
    """Returns an opaque handle (integer address).  Raises FaError on failure."""
    cfg = fa_config(ctypes.sizeof(fa_config), device, flags, wait_limit_ms, kv_splits, scratch_bytes)
    out = ctypes.c_void_p()
    st = load().fa_create(ctypes.byref(out), ctypes.byref(cfg))
    if st != FA_OK:
        raise FaError(st, "fa_create")
    return out.value


def fa_forward(h, Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale, stream=0) -> int:
    """Raw call with device pointers as integers; returns the status code."""
    return load().fa_forward(h, Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv,
                             int(bool(causal)), float(scale), stream)


def fa_forward_strided(h, Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale,
                       q_strides, k_strides, v_strides, o_strides, stream=0) -> int:
    """Raw call with device pointers and (batch, head, row) strides in elements; returns the status code."""
    arr = [(ctypes.c_int64 * 3)(*[int(x) for x in st]) for st in (q_strides, k_strides, v_strides, o_strides)]
    return load().fa_forward_strided(h, Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv, int(bool(causal)), float(scale),
                                     arr[0], arr[1], arr[2], arr[3], stream)


def fa_forward_varlen(h, Q, K, V, O, lse, cu_seqlens_q, cu_seqlens_k, B, total_q, total_k, max_sq,
                      Hq, Hkv, dqk, dv, causal, scale, stream=0) -> int:
    """Raw call on packed [total, H, d] device tensors with device int32 offsets; returns the status code."""
    return load().fa_forward_varlen(h, Q, K, V, O, lse, cu_seqlens_q, cu_seqlens_k, B, total_q, total_k, max_sq,
                                    Hq, Hkv, dqk, dv, int(bool(causal)), float(scale), stream)


def fa_forward_fp8(h, Q8, K8, V8, q_scale, k_scale, v_scale, O, lse, B, Hq, Hkv, Sq, Sk, d, causal, scale, stream=0) -> int:
    """Raw call: e4m3 device tensors with block scales (device fp32 arrays or None); returns the status code."""
    return load().fa_forward_fp8(h, Q8, K8, V8, q_scale, k_scale, v_scale, O, lse, B, Hq, Hkv, Sq, Sk, d,
                                 int(bool(causal)), float(scale), stream)


def fa_plan(num_sms, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, *, varlen=False, flags=0, kv_splits=0, scratch_bytes=0) -> dict:
    """What the library would launch for this problem on a device with `num_sms` SMs (no GPU needed)."""
    cfg = fa_config(ctypes.sizeof(fa_config), -1, flags, 0, kv_splits, scratch_bytes)
    out = fa_plan_info()
    st = load().fa_plan(num_sms, ctypes.byref(cfg), int(bool(varlen)), B, Hq, Hkv, Sq, Sk, dqk, dv, int(bool(causal)),
                        ctypes.byref(out))
    if st != FA_OK:
        raise FaError(st, "fa_plan")
    return {"kernel": out.kernel.decode(), "kv_splits": out.kv_splits, "ctas": out.ctas, "heads_per_tile": out.heads_per_tile,
            "estimate_pair_us": out.estimate_pair_us, "estimate_stream_us": out.estimate_stream_us}


def fa_forward_host(h, Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale, stream=0) -> int:
    """Raw call with HOST pointers as integers; returns the status code."""
    return load().fa_forward_host(h, Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv,
                                  int(bool(causal)), float(scale), stream)


def fa_last_status(h):
    """(status, detail) of the device-side status word; clears it."""
    detail = ctypes.c_uint32(0)
    st = load().fa_last_status(h, ctypes.byref(detail))
    return st, detail.value


def fa_destroy(h) -> int:
    return load().fa_destroy(h)


def fa_launch_count(h) -> int:
    return int(load().fa_launch_count(h))


def fa_forward_split_noalloc(Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale, kv_splits, stream=0) -> int:
    """Raw call of the allocation-free split-KV entry point (device pointers as integers, no handle).

    For callers that may not allocate: the split-KV partials live in a fixed 8 MiB array inside
    the library instead of a handle's scratch buffer.  Returns the status code.
    """
    return load().fa_forward_split_noalloc(Q, K, V, O, lse, B, Hq, Hkv, Sq, Sk, dqk, dv,
                                           int(bool(causal)), float(scale), int(kv_splits), stream)


def fa_debug_set_drop_v_load(h, enabled) -> int:
    return int(load().fa_debug_set_drop_v_load(h, int(bool(enabled))))


def fa_noalloc_scratch_bytes() -> int:
    return int(load().fa_noalloc_scratch_bytes())


def fa_noalloc_last_status():
    """(status, wait site) of the allocation-free calls on the current device since the last query; synchronises."""
    detail = ctypes.c_uint32(0)
    st = load().fa_noalloc_last_status(ctypes.byref(detail))
    return int(st), int(detail.value)


def fa_last_kv_splits(h) -> int:
    return int(load().fa_last_kv_splits(h))


def fa_last_kernel_name(h) -> str:
    return load().fa_last_kernel_name(h).decode()


def forward(h, q, k, v, *, causal: bool, scale: float = 0.0, out=None, lse=None, want_lse=True):
    """Attention forward on torch CUDA tensors (bf16, logical shape [B,H,S,d]); returns (O, lse).

    Contiguous tensors go through fa_forward.  Views with other strides (say a [B,S,H,d] buffer
    permuted to [B,H,S,d]) go through fa_forward_strided when their last dimension is contiguous;
    `out`, when not given, then takes q's memory layout.
    """
    import torch
    for t in (q, k, v):
        if t.dtype != torch.bfloat16 or not t.is_cuda or t.dim() != 4:
            raise ValueError("q, k, v must be 4-D bf16 CUDA tensors")
    B, Hq, Sq, dqk = q.shape
    _, Hkv, Sk, dv = v.shape
    dense = all(t.is_contiguous() for t in (q, k, v)) and (out is None or out.is_contiguous())
    if out is None:
        if dense:
            out = torch.empty((B, Hq, Sq, dv), dtype=torch.bfloat16, device=q.device)
        else:   # same dimension order in memory as q
            order = sorted(range(3), key=lambda i: -q.stride(i)) + [3]
            shape = (B, Hq, Sq, dv)
            buf = torch.empty([shape[i] for i in order], dtype=torch.bfloat16, device=q.device)
            out = buf.permute([order.index(i) for i in range(4)])
    if lse is None and want_lse:
        lse = torch.empty((B, Hq, Sq), dtype=torch.float32, device=q.device)
    stream = torch.cuda.current_stream(q.device).cuda_stream
    lse_ptr = lse.data_ptr() if lse is not None else None
    if dense:
        st = fa_forward(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse_ptr,
                        B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale, stream)
    else:
        for t in (q, k, v, out):
            if t.stride(3) != 1:
                raise ValueError("the last dimension must be contiguous")
        st = fa_forward_strided(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse_ptr,
                                B, Hq, Hkv, Sq, Sk, dqk, dv, causal, scale,
                                q.stride()[:3], k.stride()[:3], v.stride()[:3], out.stride()[:3], stream)
    if st != FA_OK:
        raise FaError(st, "fa_forward")
    return out, lse


def forward_varlen(h, q, k, v, cu_seqlens_q, cu_seqlens_k, max_sq: int, *, causal: bool, scale: float = 0.0,
                   want_lse=True):
    """Packed variable-length batch: q [total_q,Hq,d], k/v [total_k,Hkv,d] bf16 CUDA tensors, int32 CUDA
    offset tensors of B+1 entries.  Returns (O [total_q,Hq,dv], lse [Hq,total_q])."""
    import torch
    for t in (q, k, v):
        if t.dtype != torch.bfloat16 or not t.is_cuda or not t.is_contiguous() or t.dim() != 3:
            raise ValueError("q, k, v must be contiguous 3-D bf16 CUDA tensors")
    for t in (cu_seqlens_q, cu_seqlens_k):
        if t.dtype != torch.int32 or not t.is_cuda or not t.is_contiguous() or t.dim() != 1:
            raise ValueError("cu_seqlens must be contiguous 1-D int32 CUDA tensors")
    total_q, Hq, dqk = q.shape
    total_k, Hkv, dv = v.shape
    B = cu_seqlens_q.numel() - 1
    out = torch.empty((total_q, Hq, dv), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((Hq, total_q), dtype=torch.float32, device=q.device) if want_lse else None
    st = fa_forward_varlen(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(),
                           lse.data_ptr() if lse is not None else None,
                           cu_seqlens_q.data_ptr(), cu_seqlens_k.data_ptr(), B, total_q, total_k, int(max_sq),
                           Hq, Hkv, dqk, dv, causal, scale, torch.cuda.current_stream(q.device).cuda_stream)
    if st != FA_OK:
        raise FaError(st, "fa_forward_varlen")
    return out, lse


def forward_fp8(h, q8, k8, v8, q_scale, k_scale, v_scale, *, causal: bool, scale: float = 0.0, want_lse=True):
    """Block-scaled e4m3 attention on torch CUDA tensors: q8/k8/v8 uint8 (or float8_e4m3fn) [B,H,S,d]
    with d = 64 or 128 (or q8/k8 with d = 192 and v8 with 128), scales fp32 CUDA tensors or None.  Returns (O bf16 [B,Hq,Sq,d], lse fp32 [B,Hq,Sq])."""
    import torch
    for t in (q8, k8, v8):
        if t.element_size() != 1 or not t.is_cuda or not t.is_contiguous() or t.dim() != 4:
            raise ValueError("q8, k8, v8 must be contiguous 4-D one-byte CUDA tensors")
    B, Hq, Sq, d = q8.shape
    _, Hkv, Sk, _ = k8.shape
    dv = 128 if d == 192 else d                 # the 192/128 shapes: V and O have head size 128
    if v8.shape[-1] != dv:
        raise ValueError("v8 must have head size %d" % dv)
    n_qt, n_kt = (Sq + 127) // 128, (Sk + 127) // 128
    for t, shape in ((q_scale, (B, Hq, n_qt)), (k_scale, (B, Hkv, n_kt)), (v_scale, (B, Hkv))):
        if t is not None and (t.dtype != torch.float32 or not t.is_cuda or not t.is_contiguous() or tuple(t.shape) != shape):
            raise ValueError("scale tensors must be contiguous fp32 CUDA tensors of shape %s" % (shape,))
    out = torch.empty((B, Hq, Sq, dv), dtype=torch.bfloat16, device=q8.device)
    lse = torch.empty((B, Hq, Sq), dtype=torch.float32, device=q8.device) if want_lse else None
    ptr = lambda t: t.data_ptr() if t is not None else None
    st = fa_forward_fp8(h, q8.data_ptr(), k8.data_ptr(), v8.data_ptr(), ptr(q_scale), ptr(k_scale), ptr(v_scale),
                        out.data_ptr(), ptr(lse), B, Hq, Hkv, Sq, Sk, d, causal, scale,
                        torch.cuda.current_stream(q8.device).cuda_stream)
    if st != FA_OK:
        raise FaError(st, "fa_forward_fp8")
    return out, lse


def fa_forward_mxfp8(h, Q8, K8, V8, q_sf, k_sf, v_sf, O, lse, B, Hq, Hkv, Sq, Sk, d, causal, scale, stream=0) -> int:
    """Raw call of the MX form (e4m3 values, e8m0 scale atoms); device pointers as integers; returns the status code."""
    return load().fa_forward_mxfp8(h, Q8, K8, V8, q_sf, k_sf, v_sf, O, lse, B, Hq, Hkv, Sq, Sk, d,
                                   int(bool(causal)), float(scale), stream)


def forward_mxfp8(h, q8, k8, v8, q_sf, k_sf, v_sf, *, causal: bool, scale: float = 0.0, want_lse=True):
    """MX attention on torch CUDA tensors: q8/k8/v8 uint8 [B,H,S,d] with d = 64 or 128, scale atoms uint8
    [B,H,ceil(S/128),512] in the layout of fa_forward_mxfp8.  Returns (O bf16 [B,Hq,Sq,d], lse fp32 [B,Hq,Sq])."""
    import torch
    for t in (q8, k8, v8, q_sf, k_sf, v_sf):
        if t.element_size() != 1 or not t.is_cuda or not t.is_contiguous() or t.dim() != 4:
            raise ValueError("codes and scale atoms must be contiguous 4-D one-byte CUDA tensors")
    B, Hq, Sq, d = q8.shape
    _, Hkv, Sk, _ = k8.shape
    n_qt, n_kt = (Sq + 127) // 128, (Sk + 127) // 128
    for t, shape in ((q_sf, (B, Hq, n_qt, 512)), (k_sf, (B, Hkv, n_kt, 512)), (v_sf, (B, Hkv, n_kt, 512))):
        if tuple(t.shape) != shape:
            raise ValueError("scale atoms must have shape %s" % (shape,))
    out = torch.empty((B, Hq, Sq, d), dtype=torch.bfloat16, device=q8.device)
    lse = torch.empty((B, Hq, Sq), dtype=torch.float32, device=q8.device) if want_lse else None
    st = fa_forward_mxfp8(h, q8.data_ptr(), k8.data_ptr(), v8.data_ptr(), q_sf.data_ptr(), k_sf.data_ptr(), v_sf.data_ptr(),
                          out.data_ptr(), lse.data_ptr() if lse is not None else None, B, Hq, Hkv, Sq, Sk, d, causal, scale,
                          torch.cuda.current_stream(q8.device).cuda_stream)
    if st != FA_OK:
        raise FaError(st, "fa_forward_mxfp8")
    return out, lse
