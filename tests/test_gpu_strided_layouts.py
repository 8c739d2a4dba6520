"""fa_forward_strided: Q, K, V and O stored as [B,S,H,d], packed QKV and padded rows, against the oracle.

The oracle always sees the logical [B,H,S,d] tensors; only the GPU side's memory layout changes,
so each case also has to agree bit for bit with fa_forward on contiguous copies of the same data.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, bf16_tensor_to_f64, to_torch_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    from paper_2609_21264_b200 import binding
    h = binding.fa_create()
    yield h
    binding.fa_destroy(h)


def _status_ok(handle):
    import torch
    from paper_2609_21264_b200 import binding
    torch.cuda.synchronize()
    st, detail = binding.fa_last_status(handle)
    assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)


def _bshd(t):
    """A [B,H,S,d] view of a fresh [B,S,H,d] buffer holding the same values."""
    return t.permute(0, 2, 1, 3).contiguous().permute(0, 2, 1, 3)


CASES = [
    W.Workload("bshd_gqa_causal_d128", B=2, Hq=8, Hkv=2, Sq=333, Sk=333, dqk=128, dv=128, causal=True, scale=128 ** -0.5, seed=901),
    W.Workload("bshd_mha_d64", B=3, Hq=4, Hkv=4, Sq=200, Sk=457, dqk=64, dv=64, causal=False, scale=64 ** -0.5, seed=902),
    W.Workload("bshd_mla_like_d192", B=1, Hq=6, Hkv=6, Sq=260, Sk=260, dqk=192, dv=128, causal=True, scale=192 ** -0.5, seed=903),
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_bshd_layout_matches_oracle_and_contiguous(handle, w):
    import torch
    from paper_2609_21264_b200 import binding
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    o_c, lse_c = binding.forward(handle, q, k, v, causal=w.causal, scale=w.scale)
    qs, ks, vs = _bshd(q), _bshd(k), _bshd(v)
    assert not qs.is_contiguous()
    o_s, lse_s = binding.forward(handle, qs, ks, vs, causal=w.causal, scale=w.scale)
    _status_ok(handle)
    assert not o_s.is_contiguous() and o_s.stride(3) == 1
    assert_parity(bf16_tensor_to_f64(o_s), lse_s.double().cpu().numpy(), O_ref, lse_ref, w.name)
    assert torch.equal(o_s.contiguous().view(torch.int16), o_c.view(torch.int16))
    assert torch.equal(lse_s, lse_c)


def test_bshd_layout_serial_and_split_kernels():
    """The serial cross-check kernel and the split-KV path take the same strided tensors."""
    import torch
    from paper_2609_21264_b200 import binding
    w = CASES[0].with_(Sk=700, causal=False)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    qs, ks, vs = (_bshd(to_torch_bf16(x)) for x in (Q, K, V))
    for kw in ({"flags": binding.FA_FLAG_SERIAL_KERNEL}, {"kv_splits": 3}):
        h = binding.fa_create(**kw)
        try:
            o, lse = binding.forward(h, qs, ks, vs, causal=w.causal, scale=w.scale)
            _status_ok(h)
            assert_parity(bf16_tensor_to_f64(o), lse.double().cpu().numpy(), O_ref, lse_ref, w.name + str(kw))
        finally:
            binding.fa_destroy(h)


def test_packed_qkv_buffer(handle):
    """Q, K and V as slices of one [B, S, (Hq + 2 Hkv) * d] projection output."""
    import torch
    from paper_2609_21264_b200 import binding
    w = W.Workload("packed_qkv", B=2, Hq=8, Hkv=2, Sq=300, Sk=300, dqk=128, dv=128, causal=True, scale=128 ** -0.5, seed=904)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    packed = torch.empty((w.B, w.Sq, w.Hq + 2 * w.Hkv, 128), dtype=torch.bfloat16, device="cuda")
    packed[:, :, :w.Hq] = q.permute(0, 2, 1, 3)
    packed[:, :, w.Hq:w.Hq + w.Hkv] = k.permute(0, 2, 1, 3)
    packed[:, :, w.Hq + w.Hkv:] = v.permute(0, 2, 1, 3)
    qs = packed[:, :, :w.Hq].permute(0, 2, 1, 3)
    ks = packed[:, :, w.Hq:w.Hq + w.Hkv].permute(0, 2, 1, 3)
    vs = packed[:, :, w.Hq + w.Hkv:].permute(0, 2, 1, 3)
    o, lse = binding.forward(handle, qs, ks, vs, causal=True, scale=w.scale)
    _status_ok(handle)
    assert_parity(bf16_tensor_to_f64(o), lse.double().cpu().numpy(), O_ref, lse_ref, w.name)


def test_padded_rows_and_untouched_gaps(handle):
    """Row stride larger than the head size: the padding of O must not be written."""
    import torch
    from paper_2609_21264_b200 import binding
    w = W.Workload("padded_rows", B=1, Hq=2, Hkv=1, Sq=150, Sk=280, dqk=64, dv=64, causal=False, scale=64 ** -0.5, seed=905)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)

    def padded(t):
        buf = torch.zeros(t.shape[:3] + (t.shape[3] + 8,), dtype=torch.bfloat16, device="cuda")
        buf[..., :t.shape[3]] = t
        return buf[..., :t.shape[3]]

    q, k, v = (padded(to_torch_bf16(x)) for x in (Q, K, V))
    obuf = torch.full((w.B, w.Hq, w.Sq, w.dv + 8), 7.0, dtype=torch.bfloat16, device="cuda")
    o, lse = binding.forward(handle, q, k, v, causal=False, scale=w.scale, out=obuf[..., :w.dv])
    _status_ok(handle)
    assert_parity(bf16_tensor_to_f64(o), lse.double().cpu().numpy(), O_ref, lse_ref, w.name)
    assert (obuf[..., w.dv:] == 7.0).all()


def test_bad_strides_are_refused(handle):
    import torch
    from paper_2609_21264_b200 import binding
    t = torch.zeros((1, 1, 128, 64), dtype=torch.bfloat16, device="cuda")
    o = torch.zeros_like(t)
    good = (128 * 64, 128 * 64, 64)
    args = (handle, t.data_ptr(), t.data_ptr(), t.data_ptr(), o.data_ptr(), None, 1, 1, 1, 128, 128, 64, 64, False, 0.0)
    assert binding.fa_forward_strided(*args, good, good, good, good) == binding.FA_OK
    torch.cuda.synchronize()
    for bad in ((128 * 64, 128 * 64, 60), (128 * 64, 128 * 64 + 4, 64), (0, 128 * 64, 64), (128 * 64, 128 * 64, 32)):
        assert binding.fa_forward_strided(*args, bad, good, good, good) == binding.FA_ERR_INVALID_ARG
        assert binding.fa_forward_strided(*args, good, good, good, bad) == binding.FA_ERR_INVALID_ARG
