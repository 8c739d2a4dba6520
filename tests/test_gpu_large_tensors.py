"""Tensors of more than 2^31 elements: every offset past the 32-bit range must be computed in 64 bits.

B = 33 sequences of 16384 tokens with 32 query heads of 128 columns make Q and O 2.2e9 elements
each, so all of the last batch entry lies past element 2^31 (lse, the packed-batch row offsets and
the 8-bit code tensors likewise pass the 32-bit range of their own units).  Every batch entry holds
the same seeded data (the device copies are replicas of one host-generated entry: plumbing, no
arithmetic), which gives two checks at a size no CPU implementation could cover row by row:
  * every batch entry's output equals the first one bit for bit (a wrapped or truncated offset
    would write somewhere else and leave its own rows unwritten), and
  * rows sampled from the last entry match the oracle computed on the single entry.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, to_torch_bf16, bf16_tensor_to_f64, LSE_MAX_ABS

pytestmark = pytest.mark.gpu

B, HQ, HKV, S, D = 33, 32, 8, 16384, 128
ROWS = np.asarray([(0, h, i) for h in (0, 7, 18, 31) for i in (0, 127, 128, 5000, 8191, 8192, 16255, 16256, 16383)],
                  dtype=np.int64)


def _entry(seed):
    w = W.Workload("large_entry", B=1, Hq=HQ, Hkv=HKV, Sq=S, Sk=S, dqk=D, dv=D, causal=True, scale=D ** -0.5, seed=seed)
    return w, W.make_inputs(w)


def _replicas_equal_first(t, n, what):
    import torch
    first = t[0]
    for b in range(1, n):
        assert torch.equal(t[b], first), "%s: batch entry %d differs from entry 0" % (what, b)


def test_fixed_length_batch_past_2_31_elements():
    import torch
    from paper_2609_21264_b200 import binding
    w, (Q, K, V) = _entry(1701)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=True, scale=w.scale, rows=ROWS)
    q = to_torch_bf16(Q).expand(B, HQ, S, D).contiguous()
    k = to_torch_bf16(K).expand(B, HKV, S, D).contiguous()
    v = to_torch_bf16(V).expand(B, HKV, S, D).contiguous()
    assert q.numel() > 2 ** 31
    h = binding.fa_create()
    try:
        o, lse = binding.forward(h, q, k, v, causal=True, scale=w.scale)
        torch.cuda.synchronize()
        assert binding.fa_last_status(h)[0] == binding.FA_OK
    finally:
        binding.fa_destroy(h)
    del q, k, v
    _replicas_equal_first(o.view(torch.int16), B, "O")
    _replicas_equal_first(lse.view(torch.int32), B, "lse")
    last = B - 1
    Og = bf16_tensor_to_f64(o[last, ROWS[:, 1], ROWS[:, 2]])
    lg = lse[last, ROWS[:, 1], ROWS[:, 2]].double().cpu().numpy()
    assert_parity(Og, lg, O_ref, lse_ref, "last batch entry")


def test_packed_batch_past_2_31_elements():
    import torch
    from paper_2609_21264_b200 import binding
    w, (Q, K, V) = _entry(1702)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=True, scale=w.scale, rows=ROWS)
    # [1, H, S, d] -> [S, H, d], then the sequence B times over
    pack = lambda bits: to_torch_bf16(bits)[0].transpose(0, 1).contiguous().repeat(B, 1, 1)
    q, k, v = pack(Q), pack(K), pack(V)
    assert q.numel() > 2 ** 31
    cu = (torch.arange(B + 1, dtype=torch.int64) * S).to(torch.int32).cuda()
    h = binding.fa_create()
    try:
        o, lse = binding.forward_varlen(h, q, k, v, cu, cu, S, causal=True, scale=w.scale)
        torch.cuda.synchronize()
        assert binding.fa_last_status(h)[0] == binding.FA_OK
    finally:
        binding.fa_destroy(h)
    del q, k, v
    _replicas_equal_first(o.view(torch.int16).view(B, S, HQ, D), B, "O")
    _replicas_equal_first(lse.view(torch.int32).view(HQ, B, S).transpose(0, 1), B, "lse")
    last = (B - 1) * S
    Og = bf16_tensor_to_f64(o[last + ROWS[:, 2], ROWS[:, 1]])
    lg = lse[ROWS[:, 1], last + ROWS[:, 2]].double().cpu().numpy()
    assert_parity(Og, lg, O_ref, lse_ref, "last sequence")


def test_e4m3_batch_past_2_31_codes():
    import torch
    from paper_2609_21264_b200 import binding
    w, bits = _entry(1703)
    Q, K, V = (W.bf16_bits_to_f64(x) for x in bits)
    q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
    k8, sk, Kd = W.quantize_e4m3_blocks(K, 128)
    v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
    del Q, K, V
    O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=True, scale=w.scale, rows=ROWS)
    vmax = np.abs(Vd).max(axis=(2, 3))[0]                               # [Hkv]
    del Qd, Kd, Vd
    rep = lambda a: torch.from_numpy(a).cuda().expand(B, *a.shape[1:]).contiguous()
    h = binding.fa_create()
    try:
        o, lse = binding.forward_fp8(h, rep(q8), rep(k8), rep(v8), rep(sq), rep(sk), rep(sv), causal=True, scale=w.scale)
        torch.cuda.synchronize()
        assert binding.fa_last_status(h)[0] == binding.FA_OK
    finally:
        binding.fa_destroy(h)
    assert o.numel() > 2 ** 31
    _replicas_equal_first(o.view(torch.int16), B, "O")
    _replicas_equal_first(lse.view(torch.int32), B, "lse")
    last = B - 1
    Og = bf16_tensor_to_f64(o[last, ROWS[:, 1], ROWS[:, 2]])
    lg = lse[last, ROWS[:, 1], ROWS[:, 2]].double().cpu().numpy()
    assert np.abs(lg - lse_ref).max() <= LSE_MAX_ABS
    # the 8-bit path's bound: probabilities rounded to e4m3 (2^-4 relative) against the largest |V| of the head
    bound = 2.0 ** -4 * vmax[ROWS[:, 1] // (HQ // HKV)][:, None] + 2.0 ** -8 * np.abs(O_ref) + 1e-3
    assert (np.abs(Og - O_ref) <= bound).all()


@pytest.mark.parametrize("eight_bit", [False, True], ids=["bf16", "e4m3"])
def test_decode_step_over_a_kv_cache_past_2_31_elements(eight_bit):
    """One query per sequence against 65 x 8 x 32768 cached keys of 128 columns (2.2e9 elements each for
    K and V): grouped heads share a query tile and the K/V range is split, so the partials and the merge
    kernel are on the path too."""
    import torch
    from paper_2609_21264_b200 import binding
    nb, sk = 65, 32768
    w = W.Workload("large_decode_entry", B=1, Hq=HQ, Hkv=HKV, Sq=1, Sk=sk, dqk=D, dv=D, causal=False, scale=D ** -0.5,
                   seed=1704)
    bits = W.make_inputs(w)
    h = binding.fa_create()
    try:
        if eight_bit:
            Q, K, V = (W.bf16_bits_to_f64(x) for x in bits)
            q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
            k8, sk_, Kd = W.quantize_e4m3_blocks(K, 128)
            v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
            O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=False, scale=w.scale)
            vmax = np.abs(Vd).max(axis=(2, 3))[0]
            rep = lambda a: torch.from_numpy(a).cuda().expand(nb, *a.shape[1:]).contiguous()
            k_dev = rep(k8)
            o, lse = binding.forward_fp8(h, rep(q8), k_dev, rep(v8), rep(sq), rep(sk_), rep(sv), causal=False, scale=w.scale)
        else:
            O_ref, lse_ref = oracle.attention(*bits, causal=False, scale=w.scale)
            q = to_torch_bf16(bits[0]).expand(nb, HQ, 1, D).contiguous()
            k_dev = to_torch_bf16(bits[1]).expand(nb, HKV, sk, D).contiguous()
            v = to_torch_bf16(bits[2]).expand(nb, HKV, sk, D).contiguous()
            o, lse = binding.forward(h, q, k_dev, v, causal=False, scale=w.scale)
        torch.cuda.synchronize()
        assert binding.fa_last_status(h)[0] == binding.FA_OK
        assert k_dev.numel() > 2 ** 31
    finally:
        binding.fa_destroy(h)
    _replicas_equal_first(o.view(torch.int16), nb, "O")
    _replicas_equal_first(lse.view(torch.int32), nb, "lse")
    Og, lg = bf16_tensor_to_f64(o[nb - 1:]), lse[nb - 1:].double().cpu().numpy()
    if eight_bit:
        assert np.abs(lg - lse_ref).max() <= LSE_MAX_ABS
        bound = 2.0 ** -4 * np.repeat(vmax, HQ // HKV)[None, :, None, None] + 2.0 ** -8 * np.abs(O_ref) + 1e-3
        assert (np.abs(Og - O_ref) <= bound).all()
    else:
        assert_parity(Og, lg, O_ref, lse_ref, "last batch entry")
