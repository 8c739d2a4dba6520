"""Work and traffic counts of the attention forward pass, and the roofline that bounds it.

The throughput metric is the paper's effective-GEMM throughput (Section 5.1,
the equation defining P_effGEMM): 2*H*Lq*Lk*(dk+dv) / T.  The paper counts the
full Lq*Lk rectangle even for causal runs; `flops_paper` keeps that convention
so numbers can sit beside the paper's, while `flops_algorithmic` counts visible
(query, key) pairs only and is the one used for roofline fractions.
"""
from __future__ import annotations


def visible_pairs(Sq: int, Sk: int, causal: bool) -> int:
    """Number of (i, j) pairs with key j visible to query i, per head."""
    if not causal:
        return Sq * Sk
    off = Sk - Sq
    total = 0
    # row i sees min(Sk, max(0, i + off + 1)) keys
    lo = max(0, -off)               # first row with at least one key
    hi = min(Sq, Sk - off)          # rows below hi see all Sk keys
    if hi > lo:
        first = lo + off + 1
        last = hi - 1 + off + 1
        total += (first + last) * (hi - lo) // 2
    if Sq > max(hi, lo):
        total += (Sq - max(hi, lo)) * Sk
    return total


def flops_paper(B, Hq, Sq, Sk, dqk, dv) -> int:
    """GEMM FLOPs in the paper's convention: the full Sq*Sk rectangle."""
    return 2 * B * Hq * Sq * Sk * (dqk + dv)


def flops_algorithmic(B, Hq, Sq, Sk, dqk, dv, causal) -> int:
    """GEMM FLOPs over visible pairs only."""
    return 2 * B * Hq * visible_pairs(Sq, Sk, causal) * (dqk + dv)


def bytes_compulsory(B, Hq, Hkv, Sq, Sk, dqk, dv) -> int:
    """Q, K, V read once (bf16); O (bf16) and lse (fp32) written once."""
    elems = B * Hq * Sq * dqk + B * Hkv * Sk * dqk + B * Hkv * Sk * dv + B * Hq * Sq * dv
    return 2 * elems + 4 * B * Hq * Sq


def tflops_gemm(flops: int, seconds: float) -> float:
    return flops / seconds / 1e12


def roofline_seconds(flops_alg: int, nbytes: int, tensor_tflops: float, hbm_gbs: float):
    """(t_roof, bound): the slower of tensor time and HBM time."""
    t_tensor = flops_alg / (tensor_tflops * 1e12)
    t_hbm = nbytes / (hbm_gbs * 1e9)
    return (t_tensor, "tensor") if t_tensor >= t_hbm else (t_hbm, "hbm")
