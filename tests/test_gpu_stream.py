"""The one-query-tile-per-CTA kernel (K/V tiles streamed through both softmax warpgroups) against
the oracle, forced on for shapes of every kind, and the library's choice between the tilings.

The two warpgroups hand the row state (reference maximum and rescale factors) to each other once
per K/V tile and keep separate partial row sums, so the cases cover one, two and many K/V tiles,
odd and even counts, masked diagonals, ragged tails, rows without visible keys, growing maxima
(sigma sweep, scaled keys) and GQA.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    from paper_2609_21264_b200 import binding
    h = binding.fa_create(flags=binding.FA_FLAG_STREAM_KERNEL)
    yield h
    binding.fa_destroy(h)


def _wl(name, B, Hq, Hkv, Sq, Sk, d, causal, seed, sigma=1.0, k_mult=1.0):
    return W.Workload(name, B=B, Hq=Hq, Hkv=Hkv, Sq=Sq, Sk=Sk, dqk=d, dv=(128 if d == 192 else d), causal=causal,
                      scale=d ** -0.5, sigma=sigma, k_mult=k_mult, seed=seed)


CASES = [
    _wl("one_kv_tile", 1, 2, 2, 128, 128, 128, False, 1401),
    _wl("two_kv_tiles_ragged", 2, 4, 2, 200, 250, 128, False, 1402),
    _wl("three_kv_tiles_causal", 1, 3, 3, 333, 333, 128, True, 1403),
    _wl("many_tiles_causal_gqa", 1, 8, 2, 1100, 1100, 128, True, 1404),
    _wl("many_tiles_full_d64", 2, 4, 4, 260, 1500, 64, False, 1405),
    _wl("causal_d64_odd_tiles", 1, 5, 5, 640, 640, 64, True, 1406),
    _wl("more_queries_than_keys", 1, 2, 1, 400, 140, 128, True, 1407),
    _wl("keys_times_eight", 1, 2, 2, 384, 900, 128, True, 1408, k_mult=8.0),
    _wl("sigma_three", 1, 2, 2, 300, 700, 64, True, 1409, sigma=3.0),
    _wl("tiny", 1, 1, 1, 5, 7, 128, False, 1410),
    _wl("d192_128_causal", 1, 4, 4, 700, 700, 192, True, 1411),
    _wl("d192_128_full_ragged", 2, 2, 1, 150, 930, 192, False, 1412),
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_stream_kernel_matches_oracle(handle, w):
    from paper_2609_21264_b200 import binding
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    O, lse = run_gpu(handle, w, Q, K, V)
    assert binding.fa_last_kernel_name(handle) == "fa_fwd_stream"
    # the output bar is stated for unit-variance V; outputs and their bf16 rounding scale with sigma
    assert_parity(O / w.sigma, lse, O_ref / w.sigma, lse_ref, w.name)


def test_stream_kernel_full_size_config_1(handle):
    """Benchmark configuration 1 (the one the library routes to this kernel by default)."""
    w = W.config(0)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    O, lse = run_gpu(handle, w, Q, K, V)
    assert_parity(O, lse, O_ref, lse_ref, w.name)


def test_repeated_launches_are_bit_stable(handle):
    import torch
    from paper_2609_21264_b200 import binding
    from parity_util import to_torch_bf16
    w = CASES[3]
    Q, K, V = W.make_inputs(w)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    first = binding.forward(handle, q, k, v, causal=w.causal, scale=w.scale)[0].clone()
    outs = [binding.forward(handle, q, k, v, causal=w.causal, scale=w.scale)[0] for _ in range(20)]
    torch.cuda.synchronize()
    st, detail = binding.fa_last_status(handle)
    assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)
    for o in outs:
        assert torch.equal(o.view(torch.int16), first.view(torch.int16))


SPLIT_CASES = [
    _wl("split_decode_like", 1, 8, 2, 128, 4000, 128, False, 1421),
    _wl("split_single_row_queries", 2, 4, 4, 1, 3000, 128, False, 1422),
    _wl("split_causal_short_q", 1, 4, 4, 100, 2500, 64, True, 1423),
    _wl("split_d192", 1, 2, 2, 130, 2100, 192, False, 1424),
]


@pytest.mark.parametrize("w", SPLIT_CASES, ids=[w.name for w in SPLIT_CASES])
@pytest.mark.parametrize("splits", [0, 3, 7])
def test_stream_kernel_split_kv(w, splits):
    """K/V range cut over several CTAs of the stream kernel and merged by the combine kernel (0 = library's choice)."""
    from paper_2609_21264_b200 import binding
    h = binding.fa_create(flags=binding.FA_FLAG_STREAM_KERNEL, kv_splits=splits)
    try:
        Q, K, V = W.make_inputs(w)
        O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
        O, lse = run_gpu(h, w, Q, K, V)
        assert binding.fa_last_kernel_name(h) == "fa_fwd_stream"
        assert binding.fa_last_kv_splits(h) > 1
        assert_parity(O, lse, O_ref, lse_ref, w.name)
    finally:
        binding.fa_destroy(h)


def test_choice_between_tilings():
    """Small grids and decode-like shapes (with split-KV) go to the stream kernel, full grids to the pair kernel."""
    import torch
    from paper_2609_21264_b200 import binding
    h = binding.fa_create()
    try:
        for (B, H, Sq, Sk, causal, expect, split) in ((1, 8, 1024, 1024, True, "fa_fwd_stream", False),
                                                       (1, 32, 128, 32768, False, "fa_fwd_stream", True),
                                                       (1, 32, 2048, 2048, True, "fa_fwd_pair", False),
                                                       (1, 12, 2048, 2048, False, "fa_fwd_pair", False)):
            q = torch.zeros((B, H, Sq, 128), dtype=torch.bfloat16, device="cuda")
            k = torch.zeros((B, H, Sk, 128), dtype=torch.bfloat16, device="cuda")
            binding.forward(h, q, k, k, causal=causal)
            torch.cuda.synchronize()
            assert binding.fa_last_kernel_name(h) == expect, (B, H, Sq, Sk)
            if split:
                assert binding.fa_last_kv_splits(h) > 1, (B, H, Sq, Sk)
    finally:
        binding.fa_destroy(h)
