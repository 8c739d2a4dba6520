"""Split-KV (Algorithm 2's spatial decomposition with the corrected merge) against the fp64 oracle."""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, run_gpu

pytestmark = pytest.mark.gpu


def _wl(name, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, seed=21, k_mult=1.0):
    return W.Workload(name, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, dqk ** -0.5, 1.0, k_mult, seed)


SHAPES = [
    _wl("decode_like_gqa", 1, 8, 2, 3, 4000, 128, 128, True),
    _wl("one_tile_long_kv", 2, 4, 4, 128, 2048, 128, 128, False),
    _wl("causal_square", 1, 2, 2, 1024, 1024, 128, 128, True),          # splits beyond the diagonal are empty
    _wl("ragged_sq_gt_sk", 1, 2, 1, 333, 200, 128, 128, True),          # rows without any visible key
    _wl("ragged_d64", 1, 3, 3, 257, 1300, 64, 64, False),
    _wl("ragged_d192", 1, 2, 2, 200, 777, 192, 128, True),
    _wl("sharp_rows", 1, 2, 2, 256, 1536, 128, 128, True, k_mult=4.0),
]


@pytest.mark.parametrize("splits", [2, 3, 7])
@pytest.mark.parametrize("w", SHAPES, ids=[w.name for w in SHAPES])
def test_forced_splits_match_oracle(w, splits):
    from paper_2609_21264_b200 import binding
    h = binding.fa_create(kv_splits=splits)
    try:
        Q, K, V = W.make_inputs(w)
        O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
        O, lse = run_gpu(h, w, Q, K, V)
        assert 1 < binding.fa_last_kv_splits(h) <= splits       # capped by the number of K/V tiles
        assert_parity(O, lse, O_ref, lse_ref, w.name)
    finally:
        binding.fa_destroy(h)


def test_library_splits_short_queries_on_its_own_and_not_long_ones():
    from paper_2609_21264_b200 import binding
    h = binding.fa_create()
    try:
        w = _wl("auto_decode", 1, 16, 4, 64, 8192, 128, 128, True)
        Q, K, V = W.make_inputs(w)
        O_ref, lse_ref = oracle.attention(Q, K, V, causal=True, scale=w.scale)
        n0 = binding.fa_launch_count(h)
        O, lse = run_gpu(h, w, Q, K, V)
        assert binding.fa_last_kv_splits(h) > 1
        assert binding.fa_launch_count(h) - n0 == 2            # attention kernel + combine kernel
        assert_parity(O, lse, O_ref, lse_ref, w.name)
        w2 = _wl("auto_long", 1, 8, 2, 4096, 4096, 128, 128, True)
        Q, K, V = W.make_inputs(w2)
        run_gpu(h, w2, Q, K, V)
        assert binding.fa_last_kv_splits(h) == 1               # enough query tiles: no split
    finally:
        binding.fa_destroy(h)


def test_splitting_can_be_switched_off_and_respects_the_scratch_size():
    from paper_2609_21264_b200 import binding
    w = _wl("auto_decode", 1, 16, 4, 64, 8192, 128, 128, True)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=True, scale=w.scale)
    for kwargs, want_one in ((dict(kv_splits=1), True), (dict(scratch_bytes=1 << 16), True),
                             (dict(kv_splits=4, scratch_bytes=4 << 20), False)):
        h = binding.fa_create(**kwargs)
        try:
            O, lse = run_gpu(h, w, Q, K, V)
            assert (binding.fa_last_kv_splits(h) == 1) == want_one, kwargs
            assert_parity(O, lse, O_ref, lse_ref, str(kwargs))
        finally:
            binding.fa_destroy(h)
