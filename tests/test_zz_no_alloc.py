"""The allocation-free split-KV entry point against the handle-based one.

`fa_forward_split_noalloc` is for callers that may not allocate device memory (a server whose
memory plan is frozen, a real-time loop, a plug-in limited to its host's buffers): it takes no
handle and keeps the split-KV partials in a fixed array inside the library.  This file is
collected last on purpose, so that a run stopping at the first failure has already run every
other test; it also passes when run alone in a fresh process (it does its own set-up).
"""
import numpy as np
import pytest

from paper_2609_21264_b200 import workloads as W
from parity_util import LSE_MAX_ABS, O_MAX_ABS, O_MEAN_ABS, bf16_tensor_to_f64, to_torch_bf16

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
