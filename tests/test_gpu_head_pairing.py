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
    assert k1 == k2 == ("fa_fwd_persistent" if persistent else ("fa_fwd_pair" if w.dqk == 128 else "fa_fwd_pipelined"))
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


# (lens_q, lens_k, Hq, Hkv, d, causal): packed batches; the last two are many single-tile sequences, which the
# plan gives to the pair kernel with paired heads instead of one CTA per head
PACKED = [
    ("mix_g4", [1, 127, 128, 129, 300, 512, 57], None, 8, 2, 128, True),
    ("cross_lengths_empty_g2_d64", [40, 0, 200, 130, 5], [333, 50, 200, 0, 700], 4, 2, 64, True),
    ("no_mask_three_tiles_g2", [300, 20, 333], None, 4, 2, 128, False),
    ("d192_g2", [260, 31, 129], None, 4, 2, 192, True),
    ("single_tiles_g4", [128, 100, 1, 77, 128, 64] * 4, None, 8, 2, 128, True),
    ("single_tiles_long_keys_g2_d64", [16, 128, 90] * 14, [700, 128, 300] * 14, 4, 2, 64, True),
]


@pytest.mark.parametrize("persistent", [False, True], ids=["per_item", "persistent"])
@pytest.mark.parametrize("name,lens_q,lens_k,Hq,Hkv,d,causal", PACKED, ids=[c[0] for c in PACKED])
def test_paired_heads_in_packed_batches(name, lens_q, lens_k, Hq, Hkv, d, causal, persistent):
    import torch
    from paper_2609_21264_b200 import binding
    if persistent and d == 192:
        pytest.skip("the persistent kernel has no 192/128 variant")
    lens_k = lens_q if lens_k is None else lens_k
    dv = 128 if d == 192 else d
    tq, tk = sum(lens_q), sum(lens_k)
    w = W.Workload("packed", B=1, Hq=Hq, Hkv=Hkv, Sq=tq, Sk=tk, dqk=d, dv=dv, causal=False, scale=d ** -0.5, seed=1650 + len(lens_q))
    Q, K, V = W.make_inputs(w)                                    # [1, H, total, d] -> [total, H, d]
    q, k, v = (np.ascontiguousarray(x[0].transpose(1, 0, 2)) for x in (Q, K, V))
    cu_q = np.concatenate([[0], np.cumsum(lens_q)]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    base = binding.FA_FLAG_NO_STREAM_KERNEL | (binding.FA_FLAG_FORCE_PERSISTENT if persistent else binding.FA_FLAG_NO_PERSISTENT)
    outs = []
    for flags in (base, base | binding.FA_FLAG_NO_HEAD_PACKING):
        h = binding.fa_create(flags=flags)
        try:
            o, lse = binding.forward_varlen(h, to_torch_bf16(q), to_torch_bf16(k), to_torch_bf16(v), torch.from_numpy(cu_q).cuda(),
                                            torch.from_numpy(cu_k).cuda(), max(lens_q), causal=causal, scale=w.scale)
            torch.cuda.synchronize()
            st, detail = binding.fa_last_status(h)
            assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)
            assert binding.fa_last_kernel_name(h) == ("fa_fwd_persistent" if persistent else ("fa_fwd_pair" if d == 128 else "fa_fwd_pipelined"))
            outs.append((o, lse))
        finally:
            binding.fa_destroy(h)
    n_q_tiles = (max(lens_q) + 127) // 128
    plan = binding.fa_plan(148, len(lens_q), Hq, Hkv, max(lens_q), max(1, tk // len(lens_k)), d, dv, causal, flags=base, varlen=True)
    paired = causal or n_q_tiles % 2 == 1
    items = (n_q_tiles * (Hq // 2) if paired else (n_q_tiles + 1) // 2 * Hq) * len(lens_q)
    assert plan["ctas"] == (min(items, 148) if persistent else items), plan
    assert torch.equal(outs[0][0].view(torch.int16), outs[1][0].view(torch.int16))
    assert torch.equal(outs[0][1], outs[1][1])
    O, L = bf16_tensor_to_f64(outs[0][0]), outs[0][1].double().cpu().numpy()
    for b, (sq, sk) in enumerate(zip(lens_q, lens_k)):
        if sq == 0:
            continue
        qs, ks = slice(cu_q[b], cu_q[b + 1]), slice(cu_k[b], cu_k[b + 1])
        O_b, L_b = O[qs].transpose(1, 0, 2)[None], L[:, qs][None]
        if sk == 0:
            assert (O_b == 0).all() and np.isneginf(L_b).all()
            continue
        sl = lambda x, s: np.ascontiguousarray(x[s].transpose(1, 0, 2))[None]
        O_ref, lse_ref = oracle.attention(sl(q, qs), sl(k, ks), sl(v, ks), causal=causal, scale=w.scale)
        assert_parity(O_b, L_b, O_ref, lse_ref, "%s seq %d (%d x %d)" % (name, b, sq, sk))

