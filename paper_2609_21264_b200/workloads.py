"""Seeded synthetic workloads shared by the tests, the benchmark and the smoke check.

This module holds the workload shapes and the input generator only -- none of
the attention arithmetic.  It depends on numpy alone, so both the CPU oracle's
tests and the CUDA path's tests can draw identical inputs from it.

Inputs are i.i.d. Gaussian, as in the paper's numerical-stability protocol
(Section 5.5: entries of Q, K, V drawn from N(0, sigma^2)), rounded to bf16 with
round-to-nearest-even.  The bf16 *bit patterns* (uint16) are the inputs of
record: the oracle widens them exactly and the GPU consumes them as they are.

The shapes stand in for the paper's Table 6 (attention shapes of public LLM
configurations, synthetic data); no dataset or trained weight is involved.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, replace

import numpy as np

DEFAULT_SEED = 20260921
_TENSOR_ID = {"Q": 1, "K": 2, "V": 3}


@dataclass(frozen=True)
class Workload:
    """One attention problem: shapes, mask mode, scale and input recipe."""
    name: str
    B: int
    Hq: int
    Hkv: int
    Sq: int
    Sk: int
    dqk: int
    dv: int
    causal: bool
    scale: float
    sigma: float = 1.0
    k_mult: float = 1.0   # K is multiplied by this (exact in bf16 for powers of two)
    seed: int = DEFAULT_SEED

    def shapes(self):
        return ((self.B, self.Hq, self.Sq, self.dqk),
                (self.B, self.Hkv, self.Sk, self.dqk),
                (self.B, self.Hkv, self.Sk, self.dv),
                (self.B, self.Hq, self.Sq, self.dv))

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _w(name, B, Hq, Hkv, S, dqk, dv, causal, k_mult=1.0, idx=0):
    return Workload(name, B, Hq, Hkv, S, S, dqk, dv, causal, 1.0 / math.sqrt(dqk),
                    1.0, k_mult, DEFAULT_SEED + idx)


# The five benchmark configurations (index = position in the baseline's list).
CONFIGS = (
    _w("bert_base_mha_s512", 1, 12, 12, 512, 64, 64, False, idx=0),
    _w("llama3_8b_gqa_s2048", 1, 32, 8, 2048, 128, 128, True, idx=1),
    _w("llama2_7b_mha_b4_s8192", 4, 32, 32, 8192, 128, 128, True, k_mult=2.0, idx=2),
    _w("deepseek_v2_mha_s4096_d192_128", 1, 128, 128, 4096, 192, 128, True, idx=3),
    _w("long_context_gqa_s131072", 1, 32, 8, 131072, 128, 128, True, idx=4),
)


# The twelve attention shapes of the paper's Table 6 (LLM configurations on XDNA 2, all B = 1,
# dv = dk), with the latency the paper prints for its fused kernel in microseconds (context for
# other hardware, never a target).
TABLE6 = (
    (_w("bert_base_s2048", 1, 12, 12, 2048, 64, 64, False, idx=10), 5775.0),
    (_w("bert_large_s2048", 1, 16, 16, 2048, 64, 64, False, idx=11), 7526.0),
    (_w("gpt2_small_s2048", 1, 12, 12, 2048, 64, 64, True, idx=12), 5810.0),
    (_w("gpt2_medium_s2048", 1, 16, 16, 2048, 64, 64, True, idx=13), 7535.0),
    (_w("gpt2_large_s2048", 1, 20, 20, 2048, 64, 64, True, idx=14), 9196.0),
    (_w("llama2_7b_s2048", 1, 32, 32, 2048, 128, 128, True, idx=15), 34201.0),
    (_w("llama3_8b_s2048", 1, 32, 8, 2048, 128, 128, True, idx=16), 34076.0),
    (_w("qwen15_05b_s32768", 1, 16, 16, 32768, 64, 64, True, idx=17), 1214700.0),
    (_w("qwen25_05b_gqa_s32768", 1, 14, 2, 32768, 64, 64, True, idx=18), 1062870.0),
    (_w("qwen15_05b_s131072", 1, 16, 16, 131072, 64, 64, True, idx=19), 18996700.0),
    (_w("deepseek_7b_s4096", 1, 32, 32, 4096, 128, 128, True, idx=20), 114443.0),
    (_w("deepseek_67b_gqa_s4096", 1, 64, 8, 4096, 128, 128, True, idx=21), 227467.0),
)


def config(index_or_name) -> Workload:
    if isinstance(index_or_name, int):
        return CONFIGS[index_or_name]
    for c in CONFIGS:
        if c.name == index_or_name:
            return c
    raise KeyError(index_or_name)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(h: np.ndarray) -> np.ndarray:
    """Exact widening of bf16 bit patterns to float64."""
    w = (np.ascontiguousarray(h, dtype=np.uint16).astype(np.uint32) << np.uint32(16))
    return w.view(np.float32).astype(np.float64)


def gaussian_bf16(shape, seed: int, tensor: str, sigma: float = 1.0, mult: float = 1.0) -> np.ndarray:
    """bf16 bit patterns of mult * bf16(sigma * N(0,1)), counter-based (Philox) per (seed, tensor)."""
    key = np.array([np.uint64(seed), np.uint64(_TENSOR_ID[tensor])], dtype=np.uint64)
    gen = np.random.Generator(np.random.Philox(key=key))
    x = gen.standard_normal(size=shape, dtype=np.float32)
    if sigma != 1.0:
        x *= np.float32(sigma)
    bits = f32_to_bf16_bits(x)
    if mult != 1.0:
        # multiply the already rounded values; exact when mult is a power of two
        y = (bits.astype(np.uint32) << np.uint32(16)).view(np.float32) * np.float32(mult)
        bits = f32_to_bf16_bits(y)
    return bits


def make_inputs(w: Workload):
    """(Q, K, V) as uint16 arrays of bf16 bit patterns with the workload's shapes."""
    qs, ks, vs, _ = w.shapes()
    Q = gaussian_bf16(qs, w.seed, "Q", w.sigma)
    K = gaussian_bf16(ks, w.seed, "K", w.sigma, w.k_mult)
    V = gaussian_bf16(vs, w.seed, "V", w.sigma)
    return Q, K, V


def sample_rows(w: Workload, n_random: int, seed: int = 0, heads=None) -> np.ndarray:
    """(b, hq, i) triples: tile-boundary rows plus random rows, for sampled checks."""
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 127, 128, 129, w.Sq // 2 - 1, w.Sq // 2, w.Sq - 1]
    fixed = sorted({i for i in fixed if 0 <= i < w.Sq})
    hs = list(range(w.Hq)) if heads is None else list(heads)
    rows = []
    for b in range(w.B):
        for h in hs:
            for i in fixed:
                rows.append((b, h, i))
    for _ in range(n_random):
        rows.append((int(rng.integers(w.B)), int(hs[int(rng.integers(len(hs)))]),
                     int(rng.integers(w.Sq))))
    return np.asarray(rows, dtype=np.int64)


def quantize_e4m3_blocks(x: np.ndarray, block_rows: int | None):
    """Block-scaled e4m3 form of a [B, H, S, d] float array (input preparation for the 8-bit path).

    One fp32 scale per (batch, head, block of `block_rows` rows), or per (batch, head) when
    `block_rows` is None: scale = amax / 448 (448 = largest finite e4m3 value; 1 for an all-zero
    block), codes = round-to-nearest-even of x / scale.  Returns (codes uint8 [B,H,S,d], scales
    float32 [B,H,n_blocks] or [B,H], dequantised float64 [B,H,S,d] = codes * scale exactly).
    """
    import torch
    B, H, S, d = x.shape
    xt = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float64))
    if block_rows is None:
        amax = xt.abs().amax(dim=(2, 3))
        scales = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax)).to(torch.float32)
        per_row = scales.double()[:, :, None, None].expand(B, H, S, 1)
    else:
        nb = (S + block_rows - 1) // block_rows
        pad = nb * block_rows - S
        xp = torch.nn.functional.pad(xt, (0, 0, 0, pad)).view(B, H, nb, block_rows * d)
        amax = xp.abs().amax(dim=3)
        scales = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax)).to(torch.float32)
        per_row = scales.double().repeat_interleave(block_rows, dim=2)[:, :, :S, None]
    codes = (xt / per_row).to(torch.float32).to(torch.float8_e4m3fn)
    deq = codes.to(torch.float64) * per_row
    return codes.view(torch.uint8).numpy(), scales.numpy(), deq.numpy()


def quantize_mx_e4m3(x: np.ndarray, along: str):
    """MX (microscaling) e4m3 form of a [B, H, S, d] float array: one e8m0 scale 2^(e - 127) per block of 32
    elements, along the columns of a row (`along="cols"`: Q and K, whose contraction runs over d) or along the rows
    of a column (`along="rows"`: V, whose contraction runs over the keys).

    The scale of a block is the smallest power of two with amax / scale <= 448 (the largest e4m3 value; 2^0 for an
    all-zero block), so nothing saturates; the codes are x / scale rounded to nearest-even e4m3.  Returns (codes uint8 [B,H,S,d],
    exponent bytes uint8 [B,H,S,d/32] or [B,H,ceil(S/32),d], dequantised float64 [B,H,S,d] = codes * scale exactly).
    """
    import torch
    B, H, S, d = x.shape
    xt = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float64))
    if along == "cols":
        blocks = xt.view(B, H, S, d // 32, 32)
        amax = blocks.abs().amax(dim=4)                                       # [B,H,S,d/32]
    elif along == "rows":
        nb = (S + 31) // 32
        xp = torch.nn.functional.pad(xt, (0, 0, 0, nb * 32 - S))
        amax = xp.view(B, H, nb, 32, d).abs().amax(dim=3)                     # [B,H,nb,d]
    else:
        raise ValueError(along)
    e = torch.where(amax > 0, torch.ceil(torch.log2(torch.clamp(amax, min=1e-300) / 448.0)), torch.zeros_like(amax))
    e = torch.clamp(e, -127.0, 127.0)
    scale = torch.pow(torch.tensor(2.0, dtype=torch.float64), e)
    if along == "cols":
        per_elem = scale.repeat_interleave(32, dim=3)                         # [B,H,S,d]
    else:
        per_elem = scale.repeat_interleave(32, dim=2)[:, :, :S, :]
    q = torch.clamp(xt / per_elem, -448.0, 448.0)
    codes = q.to(torch.float32).to(torch.float8_e4m3fn)
    deq = codes.to(torch.float64) * per_elem
    return codes.view(torch.uint8).numpy(), (e + 127.0).to(torch.uint8).numpy(), deq.numpy()


def mx_scale_atoms(exps: np.ndarray, along: str, S: int) -> np.ndarray:
    """The exponent bytes of quantize_mx_e4m3 in the layout the tensor core reads: one 512-byte atom per 128-row
    tile, [B, H, ceil(S/128), 512], byte (r % 32) * 16 + (r / 32) * 4 + kb.  `along="cols"`: r = row of the tile,
    kb = block of 32 columns; `along="rows"`: r = column, kb = block of 32 rows of the tile.  Unused bytes hold 127
    (scale 1)."""
    B, H = exps.shape[:2]
    nt = (S + 127) // 128
    atoms = np.full((B, H, nt, 32, 4, 4), 127, dtype=np.uint8)                # [.., r % 32, r / 32, kb]
    if along == "cols":
        nkb = exps.shape[3]
        pad = np.full((B, H, nt * 128, nkb), 127, dtype=np.uint8)
        pad[:, :, :S] = exps
        t = pad.reshape(B, H, nt, 4, 32, nkb)                                 # [.., r / 32, r % 32, kb]
        atoms[..., :nkb] = t.transpose(0, 1, 2, 4, 3, 5)
    else:
        d = exps.shape[3]
        pad = np.full((B, H, nt * 4, d), 127, dtype=np.uint8)
        pad[:, :, :exps.shape[2]] = exps
        t = pad.reshape(B, H, nt, 4, d // 32, 32)                             # [.., kb, c / 32, c % 32]
        atoms[:, :, :, :, :d // 32, :] = t.transpose(0, 1, 2, 5, 4, 3)
    return np.ascontiguousarray(atoms.reshape(B, H, nt, 512))
