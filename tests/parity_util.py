"""Shared helpers of the GPU parity tests: run a workload through the C ABI, compare with the oracle."""
from __future__ import annotations

import numpy as np

from paper_2609_21264_b200 import workloads as W

# Tolerances of the parity bar (bf16 output, fp32 lse), stated by the benchmark contract.
O_MAX_ABS = 2e-2
O_MEAN_ABS = 2e-3
LSE_MAX_ABS = 1e-3


def to_torch_bf16(bits: np.ndarray, device="cuda"):
    import torch
    return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)


def bf16_tensor_to_f64(t) -> np.ndarray:
    import torch
    return t.detach().to("cpu").contiguous().view(torch.int16).numpy().view(np.uint16).astype(np.uint32).__lshift__(16) \
        .view(np.float32).astype(np.float64)


def run_gpu(handle, w: W.Workload, Q, K, V, want_lse=True):
    """Run the workload on the current CUDA device through fa_forward; returns (O fp64, lse fp64)."""
    import torch
    from paper_2609_21264_b200 import binding
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    o, lse = binding.forward(handle, q, k, v, causal=w.causal, scale=w.scale, want_lse=want_lse)
    torch.cuda.synchronize()
    st, detail = binding.fa_last_status(handle)
    assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)
    return bf16_tensor_to_f64(o), (lse.double().cpu().numpy() if lse is not None else None)


def errors(O_gpu, lse_gpu, O_ref, lse_ref):
    d = np.abs(O_gpu - O_ref)
    fin = np.isfinite(lse_ref)
    out = {"o_max": float(d.max()), "o_mean": float(d.mean()),
           "lse_max": float(np.abs(lse_gpu[fin] - lse_ref[fin]).max()) if fin.any() else 0.0,
           "lse_inf_match": bool(np.array_equal(np.isneginf(lse_gpu), np.isneginf(lse_ref)))}
    return out


def assert_parity(O_gpu, lse_gpu, O_ref, lse_ref, what=""):
    e = errors(O_gpu, lse_gpu, O_ref, lse_ref)
    assert np.isfinite(O_gpu).all(), what + " non-finite O"
    assert e["o_max"] <= O_MAX_ABS, (what, e)
    assert e["o_mean"] <= O_MEAN_ABS, (what, e)
    assert e["lse_max"] <= LSE_MAX_ABS, (what, e)
    assert e["lse_inf_match"], (what, e)
    return e
