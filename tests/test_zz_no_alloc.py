"""The allocation-free split-KV entry point against the oracle and against the handle-based one.

`fa_forward_split_noalloc` is for callers that may not allocate device memory (a server whose
memory plan is frozen, a real-time loop, a plug-in limited to its host's buffers): it takes no
handle and keeps the split-KV partials in a fixed array inside the library.  This file is
collected last on purpose, so that a run stopping at the first failure has already run every
other test; it also passes when run alone in a fresh process (it does its own set-up).
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import LSE_MAX_ABS, O_MAX_ABS, O_MEAN_ABS, assert_parity, bf16_tensor_to_f64, to_torch_bf16

pytestmark = pytest.mark.gpu


def _both_paths(w, splits, handle):
    """(O, lse) from fa_forward (handle, scratch from fa_create) and from the no-alloc entry point."""
    import torch
    from paper_2609_21264_b200 import binding as b
    Q, K, V = W.make_inputs(w)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    outs = []
    for use_handle in (True, False):
        o = torch.full((w.B, w.Hq, w.Sq, w.dv), float("nan"), dtype=torch.bfloat16, device="cuda")
        lse = torch.full((w.B, w.Hq, w.Sq), float("nan"), dtype=torch.float32, device="cuda")
        stream = torch.cuda.current_stream().cuda_stream
        args = (q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr(),
                w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv, w.causal, w.scale)
        if use_handle:
            st = b.fa_forward(handle, *args, stream)
            assert b.fa_last_kv_splits(handle) > 1
        else:
            st = b.fa_forward_split_noalloc(*args, splits, stream)
        assert st == b.FA_OK, b.fa_strerror(st)
        torch.cuda.synchronize()
        outs.append((bf16_tensor_to_f64(o), lse.double().cpu().numpy()))
    return outs


def test_no_alloc_entry_point_matches_handle_path_on_two_calls_in_a_row():
    from paper_2609_21264_b200 import binding as b
    assert b.fa_noalloc_scratch_bytes() == 8 << 20
    splits = 4
    h = b.fa_create(kv_splits=splits)
    try:
        # second call: different shape and inputs, fewer rows, so stale partials of the first call
        # (the array is shared and never cleared) would show up if any slot were read unwritten
        shapes = [W.Workload("first", 1, 8, 2, 96, 4096, 128, 128, True, 128 ** -0.5, seed=31),
                  W.Workload("second", 2, 4, 4, 40, 1500, 64, 64, False, 64 ** -0.5, seed=32)]
        for w in shapes:
            (O_h, lse_h), (O_n, lse_n) = _both_paths(w, splits, h)
            assert np.isfinite(O_n).all() and np.isfinite(lse_n).all()
            d = np.abs(O_n - O_h)
            assert d.max() <= O_MAX_ABS and d.mean() <= O_MEAN_ABS, (w.name, d.max(), d.mean())
            assert np.abs(lse_n - lse_h).max() <= LSE_MAX_ABS, w.name
        st, _ = b.fa_last_status(h)
        assert st == b.FA_OK
    finally:
        b.fa_destroy(h)


def _no_alloc(w, splits, want_lse=True):
    import torch
    from paper_2609_21264_b200 import binding as b
    Q, K, V = W.make_inputs(w)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    o = torch.full((w.B, w.Hq, w.Sq, w.dv), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((w.B, w.Hq, w.Sq), float("nan"), dtype=torch.float32, device="cuda") if want_lse else None
    st = b.fa_forward_split_noalloc(q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(), lse.data_ptr() if want_lse else None,
                                    w.B, w.Hq, w.Hkv, w.Sq, w.Sk, w.dqk, w.dv, w.causal, w.scale, splits,
                                    torch.cuda.current_stream().cuda_stream)
    assert st == b.FA_OK, b.fa_strerror(st)
    torch.cuda.synchronize()
    assert b.fa_noalloc_last_status() == (b.FA_OK, 0)
    return (Q, K, V), bf16_tensor_to_f64(o), (lse.double().cpu().numpy() if want_lse else None)


# Shapes chosen for what the shared array and the split path can get wrong: later splits that are empty under a causal
# mask, a forced empty split (fewer K/V tiles than splits), the asymmetric head sizes, an odd number of query tiles,
# more queries than keys (rows with no visible key at all), and partials that fill the 8 MiB array to the last byte.
ORACLE_CASES = [
    (W.Workload("causal_multi_tile_empty_late_splits", 1, 4, 2, 384, 384, 128, 128, True, 128 ** -0.5, seed=41), 3),
    (W.Workload("one_kv_tile_two_splits", 1, 6, 3, 100, 128, 64, 64, False, 64 ** -0.5, seed=42), 2),
    (W.Workload("d192_dv128", 1, 4, 2, 200, 1000, 192, 128, True, 192 ** -0.5, seed=43), 4),
    (W.Workload("odd_number_of_query_tiles", 1, 2, 2, 300, 2100, 128, 128, False, 128 ** -0.5, seed=44), 5),
    (W.Workload("more_queries_than_keys", 1, 2, 1, 333, 200, 128, 128, True, 128 ** -0.5, seed=45), 2),
    # 2 splits x (1 x 8 x 1016) rows x 129 floats x 4 bytes = 8 388 096 bytes + ... : the largest row count that fits
    (W.Workload("partials_at_the_limit", 1, 8, 4, (8 << 20) // (2 * 8 * 129 * 4), 700, 128, 128, False, 128 ** -0.5, seed=46), 2),
]


@pytest.mark.parametrize("w,splits", ORACLE_CASES, ids=[c[0].name for c in ORACLE_CASES])
def test_no_alloc_entry_point_against_the_oracle(w, splits):
    from paper_2609_21264_b200 import binding as b
    if w.name == "partials_at_the_limit":
        need = splits * w.B * w.Hq * w.Sq * (w.dv + 1) * 4
        assert need <= b.fa_noalloc_scratch_bytes() < splits * w.B * w.Hq * (w.Sq + 1) * (w.dv + 1) * 4
    (Q, K, V), O, lse = _no_alloc(w, splits)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    assert_parity(O, lse, O_ref, lse_ref, w.name)
    if w.name == "more_queries_than_keys":
        assert np.isneginf(lse_ref).any() and (O[np.isneginf(lse_ref)] == 0).all()
    # once more without the log-sum-exp output (a NULL pointer is legal), on what the first call left in the array
    _, O2, _ = _no_alloc(w, splits, want_lse=False)
    np.testing.assert_array_equal(O, O2)


def test_no_alloc_entry_point_rejects_what_does_not_fit_and_bad_arguments():
    import torch
    from paper_2609_21264_b200 import binding as b
    t = torch.zeros(1 << 20, dtype=torch.bfloat16, device="cuda")
    p = t.data_ptr()
    # 4 splits x (1*32*4096 rows) x 129 floats = 270 MB of partials: far beyond the 8 MiB array
    assert b.fa_forward_split_noalloc(p, p, p, p, None, 1, 32, 8, 4096, 4096, 128, 128, True, 0.0, 4, 0) \
        == b.FA_ERR_UNSUPPORTED
    assert b.fa_forward_split_noalloc(p, p, p, p, None, 1, 2, 2, 64, 1024, 128, 128, False, 0.0, 1, 0) \
        == b.FA_ERR_INVALID_ARG          # kv_splits below 2
    assert b.fa_forward_split_noalloc(None, p, p, p, None, 1, 2, 2, 64, 1024, 128, 128, False, 0.0, 2, 0) \
        == b.FA_ERR_INVALID_ARG
    assert b.fa_forward_split_noalloc(p, p, p, p, None, 1, 2, 2, 64, 1024, 96, 96, False, 0.0, 2, 0) \
        == b.FA_ERR_UNSUPPORTED
    torch.cuda.synchronize()
