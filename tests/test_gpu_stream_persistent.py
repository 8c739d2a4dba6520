"""The persistent form of the stream kernel (csrc/fa_fwd_stream_persistent.cuh): one CTA per SM draws one-tile work
items from a ticket counter; the next item's Q, first K/V tiles and first scores overlap the current item's tail, and
the output is staged in a stage of the K ring.

The cases give every SM several items and cover what has to carry over from item to item: items with odd and even
numbers of K/V tiles in any order (the two S/P buffer pairs' use counts drift apart), items with a single K/V tile
(the staging stage's previous tenant is the previous item's staging tile), items without any visible key in between
(no barrier traffic at all), ragged tiles, grouped heads, all three head sizes, and several launches through one
handle (the ticket counter is back at zero after every launch).  Same arithmetic as the one-item stream kernel: the
results are equal bit for bit.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, to_torch_bf16, bf16_tensor_to_f64

pytestmark = pytest.mark.gpu


def _wl(name, B, Hq, Hkv, Sq, Sk, d, seed, causal=True):
    return W.Workload(name, B=B, Hq=Hq, Hkv=Hkv, Sq=Sq, Sk=Sk, dqk=d, dv=128 if d == 192 else d, causal=causal,
                      scale=d ** -0.5, seed=seed)


CASES = [
    _wl("d192_causal_gqa_four_tiles", 4, 32, 8, 512, 512, 192, 2301),
    _wl("d192_single_kv_tile_items", 16, 32, 32, 128, 128, 192, 2302),
    _wl("d128_causal_eight_tiles", 2, 32, 32, 1024, 1024, 128, 2303),
    _wl("d64_causal_four_tiles", 8, 16, 16, 512, 512, 64, 2304),
    _wl("d192_ragged_fewer_queries_than_keys", 2, 40, 8, 700, 1000, 192, 2305),
    _wl("d128_more_queries_than_keys_items_without_keys", 1, 52, 52, 1100, 300, 128, 2306),
    _wl("d192_no_mask_odd_tile_counts", 4, 40, 40, 384, 640, 192, 2307, causal=False),
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_persistent_stream_kernel_matches_the_oracle_and_the_one_item_kernel(w):
    import torch
    from paper_2609_21264_b200 import binding
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    h = binding.fa_create(flags=binding.FA_FLAG_STREAM_KERNEL, wait_limit_ms=500, kv_splits=1)
    h1 = binding.fa_create(flags=binding.FA_FLAG_STREAM_KERNEL | binding.FA_FLAG_NO_PERSISTENT, wait_limit_ms=500, kv_splits=1)
    try:
        for rep in range(3):            # the ticket counter is back at zero after every launch
            o, lse = binding.forward(h, q, k, v, causal=w.causal, scale=w.scale)
            torch.cuda.synchronize()
            st, site = binding.fa_last_status(h)
            assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, site)
            assert binding.fa_last_kernel_name(h) == "fa_fwd_stream_persistent"
            if rep == 0:
                assert_parity(bf16_tensor_to_f64(o), lse.double().cpu().numpy(), O_ref, lse_ref, w.name)
                first = (o.clone(), lse.clone())
            else:
                assert torch.equal(first[0], o) and torch.equal(first[1], lse)
        o1, lse1 = binding.forward(h1, q, k, v, causal=w.causal, scale=w.scale)
        torch.cuda.synchronize()
        assert binding.fa_last_kernel_name(h1) == "fa_fwd_stream"
        assert torch.equal(o1, first[0]) and torch.equal(lse1, first[1])
    finally:
        assert binding.fa_destroy(h) == binding.FA_OK
        assert binding.fa_destroy(h1) == binding.FA_OK


def test_back_to_back_launches_of_varied_shapes_equal_the_one_item_kernel():
    """Hundreds of launches through one handle without a synchronisation in between, shapes changing every 25 launches
    (the ticket counter and the tensor-map cache carry over): every result equals the one-item kernel's bit for bit
    and no wait runs out."""
    import random
    import torch
    from paper_2609_21264_b200 import binding
    rnd = random.Random(2310)
    h = binding.fa_create(wait_limit_ms=2000)
    h1 = binding.fa_create(flags=binding.FA_FLAG_NO_PERSISTENT, wait_limit_ms=2000)
    try:
        gen = torch.Generator(device="cuda").manual_seed(2310)
        persistent = 0
        for it in range(12):
            B, H = rnd.choice([1, 2, 4]), rnd.choice([32, 64, 128])
            S = rnd.choice([384, 512, 1024, 1536, 2048, 3072])
            Sk = S + rnd.choice([0, 0, 128, 700])
            causal = rnd.random() < 0.7
            q = torch.randn((B, H, S, 192), generator=gen, device="cuda").bfloat16()
            k = torch.randn((B, H, Sk, 192), generator=gen, device="cuda").bfloat16()
            v = torch.randn((B, H, Sk, 128), generator=gen, device="cuda").bfloat16()
            o_ref, l_ref = binding.forward(h1, q, k, v, causal=causal)
            for _ in range(25):
                o, l = binding.forward(h, q, k, v, causal=causal)
            torch.cuda.synchronize()
            assert binding.fa_last_status(h) == (binding.FA_OK, 0)
            persistent += binding.fa_last_kernel_name(h) == "fa_fwd_stream_persistent"
            assert torch.equal(o, o_ref) and torch.equal(l, l_ref), (it, B, H, S, Sk, causal)
        assert persistent >= 4          # the draw reaches the kernel this test is about
    finally:
        assert binding.fa_destroy(h) == binding.FA_OK
        assert binding.fa_destroy(h1) == binding.FA_OK
