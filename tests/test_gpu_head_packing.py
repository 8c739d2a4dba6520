"""Grouped-query attention with few queries per sequence: several query heads of one K/V head share
a query tile of the stream kernel (row h * Sq + i of the tile is query i of the h-th head).

Checked against the oracle for every way the packing can go wrong: group sizes whose largest
fitting divisor is the whole group, a part of it, or leaves the tile partly empty; a single query
per sequence; odd Sq (box rows that are no multiple of the 8-row swizzle period); causal masks
whose diagonal depends on the row's index inside its head; rows without a visible key; split-KV;
strided tensors; and against the unpacked launch bit for bit.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, run_gpu, to_torch_bf16, bf16_tensor_to_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    from paper_2609_21264_b200 import binding
    h = binding.fa_create()
    yield h
    binding.fa_destroy(h)


def _wl(name, B, Hq, Hkv, Sq, Sk, d, causal, seed, sigma=1.0):
    return W.Workload(name, B=B, Hq=Hq, Hkv=Hkv, Sq=Sq, Sk=Sk, dqk=d, dv=(128 if d == 192 else d), causal=causal,
                      scale=d ** -0.5, sigma=sigma, seed=seed)


# (workload, heads per tile the plan must choose)
CASES = [
    (_wl("group4_sq16_half_tile", 2, 8, 2, 16, 700, 128, False, 1501), 4),
    (_wl("group8_sq16_full_tile_causal", 1, 8, 1, 16, 1000, 128, True, 1502), 8),
    (_wl("group3_sq20_d64_causal", 2, 6, 2, 20, 333, 64, True, 1503), 3),
    (_wl("group2_sq64_full_tile_causal", 1, 4, 2, 64, 500, 128, True, 1504), 2),
    (_wl("group6_single_query_long_k", 1, 12, 2, 1, 4100, 128, False, 1505), 6),
    (_wl("group4_sq7_d192_causal", 1, 8, 2, 7, 300, 192, True, 1506), 4),
    (_wl("group4_sq33_only_two_fit", 3, 16, 4, 33, 260, 128, True, 1507), 2),
    (_wl("group2_more_queries_than_keys", 1, 4, 2, 40, 20, 128, True, 1508), 2),
    (_wl("group16_sq5_many_heads", 2, 32, 2, 5, 650, 64, False, 1509), 16),
    (_wl("group4_sq16_sigma3", 1, 8, 2, 16, 900, 128, True, 1510, sigma=3.0), 4),
]


@pytest.mark.parametrize("w,heads", CASES, ids=[c[0].name for c in CASES])
def test_packed_heads_match_oracle(handle, w, heads):
    import torch
    from paper_2609_21264_b200 import binding
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    plan = binding.fa_plan(sms, w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv, w.causal)
    assert plan["kernel"] == "fa_fwd_stream" and plan["heads_per_tile"] == heads, plan
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    O, lse = run_gpu(handle, w, Q, K, V)
    assert binding.fa_last_kernel_name(handle) == "fa_fwd_stream"
    assert binding.fa_last_kv_splits(handle) == plan["kv_splits"]
    assert_parity(O / w.sigma, lse, O_ref / w.sigma, lse_ref, w.name)


@pytest.mark.parametrize("splits", [1, 3])
def test_packed_equals_unpacked_bit_for_bit(splits):
    """A row's arithmetic does not depend on which rows share its tile: same split count, same bits."""
    import torch
    from paper_2609_21264_b200 import binding
    hp = binding.fa_create(flags=binding.FA_FLAG_STREAM_KERNEL, kv_splits=splits)
    hu = binding.fa_create(flags=binding.FA_FLAG_STREAM_KERNEL | binding.FA_FLAG_NO_HEAD_PACKING, kv_splits=splits)
    try:
        for w in (_wl("eq_full", 2, 8, 2, 24, 1300, 128, False, 1520), _wl("eq_causal_d64", 1, 6, 2, 11, 777, 64, True, 1521)):
            Q, K, V = W.make_inputs(w)
            q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
            o1, l1 = binding.forward(hp, q, k, v, causal=w.causal, scale=w.scale)
            o2, l2 = binding.forward(hu, q, k, v, causal=w.causal, scale=w.scale)
            torch.cuda.synchronize()
            assert binding.fa_last_status(hp)[0] == binding.FA_OK and binding.fa_last_status(hu)[0] == binding.FA_OK
            assert binding.fa_last_kv_splits(hp) == splits and binding.fa_last_kv_splits(hu) == splits
            assert torch.equal(o1.view(torch.int16), o2.view(torch.int16)), w.name
            assert torch.equal(l1, l2), w.name
    finally:
        binding.fa_destroy(hp)
        binding.fa_destroy(hu)


def test_packed_heads_with_strided_tensors(handle):
    """[B, S, H, d] storage: the box of heads follows the head stride of the tensor map."""
    import torch
    from paper_2609_21264_b200 import binding
    w = _wl("packed_bshd", 2, 8, 2, 12, 520, 128, True, 1530)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    q, k, v = (to_torch_bf16(x).transpose(1, 2).contiguous().transpose(1, 2) for x in (Q, K, V))
    assert not q.is_contiguous()
    o, lse = binding.forward(handle, q, k, v, causal=w.causal, scale=w.scale)
    torch.cuda.synchronize()
    assert binding.fa_last_status(handle)[0] == binding.FA_OK
    assert binding.fa_last_kernel_name(handle) == "fa_fwd_stream"
    assert_parity(bf16_tensor_to_f64(o), lse.double().cpu().numpy(), O_ref, lse_ref, w.name)


def test_repeated_packed_launches_are_bit_stable(handle):
    import torch
    from paper_2609_21264_b200 import binding
    w = _wl("packed_repeat", 1, 32, 8, 16, 8192, 128, False, 1531)
    Q, K, V = W.make_inputs(w)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    first = binding.forward(handle, q, k, v, causal=w.causal, scale=w.scale)[0].clone()
    outs = [binding.forward(handle, q, k, v, causal=w.causal, scale=w.scale)[0] for _ in range(20)]
    torch.cuda.synchronize()
    assert binding.fa_last_status(handle)[0] == binding.FA_OK
    for o in outs:
        assert torch.equal(o.view(torch.int16), first.view(torch.int16))
