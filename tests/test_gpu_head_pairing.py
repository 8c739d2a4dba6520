"""Causal grouped-query attention on the pair tilings: a CTA's two query tiles are the SAME query
tile of two adjacent heads of a K/V group (equal numbers of K/V tiles, no round that one tile runs
alone) instead of two adjacent query tiles of one head.

A tile's arithmetic does not depend on which tile shares its CTA, so the result has to be the
unpaired launch's bit for bit; the cases cover ragged and odd numbers of query tiles, more queries
than keys (tiles without a visible key), Sq != Sk, several batches and K/V heads, group sizes 2, 4
and 6, all head sizes, the persistent kernel and the 8-bit path, each also against the oracle.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, to_torch_bf16, bf16_tensor_to_f64

pytestmark = pytest.mark.gpu


def _wl(name, B, Hq, Hkv, Sq, Sk, d, seed, causal=True):
    return W.Workload(name, B=B, Hq=Hq, Hkv=Hkv, Sq=Sq, Sk=Sk, dqk=d, dv=(128 if d == 192 else d), causal=causal,
                      scale=d ** -0.5, seed=seed)


CASES = [
    _wl("g4_ragged_odd_tiles", 2, 8, 2, 333, 333, 128, 1601),
    _wl("g2_more_queries_than_keys", 1, 4, 2, 400, 140, 128, 1602),
    _wl("g6_d64", 1, 12, 2, 700, 700, 64, 1603),
    _wl("g2_single_tile", 1, 2, 1, 128, 128, 128, 1604),
    _wl("g2_d192", 1, 4, 2, 300, 300, 192, 1605),
    _wl("g4_fewer_queries_than_keys", 3, 16, 4, 260, 900, 128, 1606),
    _wl("g4_llama_like_s1024", 2, 16, 4, 1024, 1024, 128, 1607),
    # no mask: paired for an odd number of query tiles (the last tile of a head would be alone in its CTA)
    _wl("g4_no_mask_three_tiles", 4, 16, 4, 333, 500, 128, 1608, causal=False),
    _wl("g2_no_mask_five_tiles_d64", 3, 12, 6, 600, 600, 64, 1609, causal=False),
]


def _run(flags, w, Q, K, V):
    import torch
    from paper_2609_21264_b200 import binding
    h = binding.fa_create(flags=flags)
    try:
        o, lse = binding.forward(h, to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V), causal=w.causal, scale=w.scale)
        torch.cuda.synchronize()
        st, detail = binding.fa_last_status(h)
        assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)
        return o, lse, binding.fa_last_kernel_name(h)
    finally:
        binding.fa_destroy(h)


@pytest.mark.parametrize("persistent", [False, True], ids=["per_item", "persistent"])
@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_paired_heads_equal_the_unpaired_launch_and_the_oracle(w, persistent):
    import torch
    from paper_2609_21264_b200 import binding
    if persistent and w.dqk == 192:
        pytest.skip("the persistent kernel has no 192/128 variant")
    base = binding.FA_FLAG_NO_STREAM_KERNEL | (binding.FA_FLAG_FORCE_PERSISTENT if persistent else binding.FA_FLAG_NO_PERSISTENT)
    Q, K, V = W.make_inputs(w)
    o1, l1, k1 = _run(base, w, Q, K, V)
    o2, l2, k2 = _run(base | binding.FA_FLAG_NO_HEAD_PACKING, w, Q, K, V)
    assert k1 == k2 == ("fa_fwd_persistent" if persistent else "fa_fwd_pipelined")
    sms = torch.cuda.get_device_properties(0).multi_processor_count
    n_q_tiles = (w.Sq + 127) // 128
    plan = binding.fa_plan(sms, w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv, w.causal, flags=base)
    if plan["kv_splits"] == 1:      # (a split K/V range keeps the pairs of adjacent query tiles)
        assert plan["ctas"] == min(n_q_tiles * (w.Hq // 2) * w.B, sms if persistent else 1 << 30), plan     # one item per tile and pair of heads
    assert torch.equal(o1.view(torch.int16), o2.view(torch.int16))
    assert torch.equal(l1, l2)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    assert_parity(bf16_tensor_to_f64(o1), l1.double().cpu().numpy(), O_ref, lse_ref, w.name)


def test_paired_heads_on_the_8_bit_path():
    import torch
    from paper_2609_21264_b200 import binding
    for d in (64, 128):
        w = _wl("fp8_pairing_d%d" % d, 2, 8, 2, 450, 450, d, 1610 + d)
        Q, K, V = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
        q8, sq, _ = W.quantize_e4m3_blocks(Q, 128)
        k8, sk, _ = W.quantize_e4m3_blocks(K, 128)
        v8, sv, _ = W.quantize_e4m3_blocks(V, None)
        dev = lambda a: torch.from_numpy(a).cuda()
        outs = []
        for flags in (binding.FA_FLAG_NO_STREAM_KERNEL, binding.FA_FLAG_NO_STREAM_KERNEL | binding.FA_FLAG_NO_HEAD_PACKING):
            h = binding.fa_create(flags=flags)
            try:
                o, lse = binding.forward_fp8(h, dev(q8), dev(k8), dev(v8), dev(sq), dev(sk), dev(sv), causal=True, scale=w.scale)
                torch.cuda.synchronize()
                assert binding.fa_last_status(h)[0] == binding.FA_OK and binding.fa_last_kernel_name(h) == "fa_fwd_fp8"
                outs.append((o, lse))
            finally:
                binding.fa_destroy(h)
        assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
        assert torch.equal(outs[0][1], outs[1][1])
