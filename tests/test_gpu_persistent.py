"""The persistent kernel (one CTA per SM walking a list of work items) against the oracle and,
bit for bit, against the one-item-per-CTA kernel: both run the same arithmetic in the same order.

Shapes are chosen so that CTAs process several items each (more items than SMs), including items
whose second query tile does not exist, tiles without any visible key, and ragged tails.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, bf16_tensor_to_f64, to_torch_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handles():
    from paper_2609_21264_b200 import binding
    hs = {"persistent": binding.fa_create(flags=binding.FA_FLAG_FORCE_PERSISTENT),
          "per_item": binding.fa_create(flags=binding.FA_FLAG_NO_PERSISTENT | binding.FA_FLAG_NO_STREAM_KERNEL)}
    yield hs
    for h in hs.values():
        binding.fa_destroy(h)


def _wl(name, B, Hq, Hkv, Sq, Sk, d, causal, seed):
    return W.Workload(name, B=B, Hq=Hq, Hkv=Hkv, Sq=Sq, Sk=Sk, dqk=d, dv=d, causal=causal, scale=d ** -0.5, seed=seed)


CASES = [
    _wl("many_items_causal_d128", 2, 40, 8, 600, 600, 128, True, 1201),      # 240 items, odd tile count
    _wl("many_items_full_d128", 1, 160, 160, 300, 417, 128, False, 1202),    # 320 items, ragged K/V tail
    _wl("many_items_causal_d64", 3, 64, 16, 512, 512, 64, True, 1203),       # 384 items
    _wl("more_queries_than_keys", 1, 150, 150, 400, 140, 128, True, 1204),   # tiles with no visible key
    _wl("fewer_items_than_sms", 1, 4, 2, 700, 700, 128, True, 1205),         # 12 items: short grid
    _wl("single_tile_items", 1, 300, 300, 100, 260, 64, False, 1206),        # tile 1 never exists
    # head size 64: the per-item kernel keeps P in TMEM columns of its own and issues score blocks ahead of
    # the PV products, the persistent kernel does not; items long enough for the hand-offs to wrap many times
    _wl("long_causal_items_d64", 2, 12, 12, 2048, 2048, 64, True, 1207),     # up to 16 K/V tiles, tile 0 one short of tile 1
    _wl("long_full_items_d64", 1, 20, 4, 1100, 2300, 64, False, 1208),       # 18 K/V tiles, ragged tails
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_persistent_matches_oracle_and_per_item_kernel(handles, w):
    import torch
    from paper_2609_21264_b200 import binding
    Q, K, V = W.make_inputs(w)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    out = {}
    for name, h in handles.items():
        o, lse = binding.forward(h, q, k, v, causal=w.causal, scale=w.scale)
        torch.cuda.synchronize()
        st, detail = binding.fa_last_status(h)
        assert st == binding.FA_OK, "%s: device status %d (site 0x%x)" % (name, st, detail)
        out[name] = (o, lse)
    assert binding.fa_last_kernel_name(handles["persistent"]) == "fa_fwd_persistent"
    assert binding.fa_last_kernel_name(handles["per_item"]) == ("fa_fwd_pair" if w.dqk == 128 else "fa_fwd_pipelined")
    o_p, lse_p = out["persistent"]
    o_i, lse_i = out["per_item"]
    assert torch.equal(o_p.view(torch.int16), o_i.view(torch.int16))
    assert torch.equal(lse_p, lse_i)
    heads = sorted({0, w.Hq // 2, w.Hq - 1})
    rows = np.array([(b, h, i) for b in range(w.B) for h in heads for i in range(w.Sq)], dtype=np.int64)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale, rows=rows)
    O = bf16_tensor_to_f64(o_p)[rows[:, 0], rows[:, 1], rows[:, 2]]
    L = lse_p.double().cpu().numpy()[rows[:, 0], rows[:, 1], rows[:, 2]]
    assert_parity(O, L, O_ref, lse_ref, w.name)


def test_repeated_launches_reuse_state_cleanly(handles):
    """Back-to-back launches (dependent launch overlaps their tails) keep giving the same bits."""
    import torch
    from paper_2609_21264_b200 import binding
    w = CASES[0]
    Q, K, V = W.make_inputs(w)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    h = handles["persistent"]
    first, _ = binding.forward(h, q, k, v, causal=w.causal, scale=w.scale)
    first = first.clone()
    outs = [binding.forward(h, q, k, v, causal=w.causal, scale=w.scale)[0] for _ in range(8)]
    torch.cuda.synchronize()
    for o in outs:
        assert torch.equal(o.view(torch.int16), first.view(torch.int16))


def test_default_choice_by_shape():
    from paper_2609_21264_b200 import binding
    import torch
    h = binding.fa_create()
    try:
        for (B, H, S, expect) in ((8, 32, 1024, "fa_fwd_persistent"), (1, 32, 2048, "fa_fwd_pair"),
                                  (1, 12, 512, "fa_fwd_stream"), (1, 64, 16384, "fa_fwd_persistent"),
                                  (1, 16, 32768, "fa_fwd_pair")):     # items of 256 K/V tiles: past the persistent kernel's range
            q = torch.zeros((B, H, S, 128), dtype=torch.bfloat16, device="cuda")
            binding.forward(h, q, q, q, causal=True)
            torch.cuda.synchronize()
            assert binding.fa_last_kernel_name(h) == expect, (B, H, S)
    finally:
        binding.fa_destroy(h)
