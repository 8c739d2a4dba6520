"""fa_forward_host on problems of 256 MiB and more: the call is cut into chunks of whole (batch, K/V head) units whose
copies in and out overlap the other chunks' kernels on copy streams of the handle.

A chunk is the same attention problem on a slice of the heads or of the batch, so the result has to equal the
device-buffer entry's on the whole problem bit for bit (the kernels a chunk's shape may select instead are
bit-identical at this head size), and sampled rows have to match the oracle.  The three shapes reach the three ways of
cutting: K/V-head ranges of a single batch entry, whole batch entries, and head ranges within several batch entries
(where the last range of each entry is shorter); the third also runs without an lse buffer.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, run_gpu

pytestmark = pytest.mark.gpu

CASES = [
    # name, B, Hq, Hkv, S  (d = 128, causal): total bytes of Q, K, V, O, lse
    ("head_ranges_of_one_batch_entry", 1, 32, 8, 16384),       # 340 MB -> 2 chunks of 4 K/V heads
    ("whole_batch_entries", 3, 16, 4, 16384),                  # 510 MB -> 3 chunks of one batch entry
    ("head_ranges_in_two_batch_entries", 2, 24, 3, 16384),     # 455 MB -> 3 chunks wanted, 2 per entry: K/V heads 2 + 1
]


@pytest.mark.parametrize("case", CASES, ids=[c[0] for c in CASES])
def test_chunked_host_call_equals_the_device_call_and_the_oracle(case):
    import torch
    from paper_2609_21264_b200 import binding
    name, B, Hq, Hkv, S = case
    w = W.Workload(name, B=B, Hq=Hq, Hkv=Hkv, Sq=S, Sk=S, dqk=128, dv=128, causal=True, scale=128 ** -0.5, seed=3100 + B)
    Q, K, V = W.make_inputs(w)
    h = binding.fa_create()
    try:
        O_dev, lse_dev = run_gpu(h, w, Q, K, V)                   # device buffers, one launch
        # pinned host buffers: the copies are asynchronous and overlap the kernels
        pin = lambda a: torch.from_numpy(a.view(np.int16)).pin_memory()
        q, k, v = pin(Q), pin(K), pin(V)
        o = torch.empty((B, Hq, S, 128), dtype=torch.int16).pin_memory()
        lse = torch.empty((B, Hq, S), dtype=torch.float32).pin_memory()
        stream = torch.cuda.current_stream().cuda_stream
        for want_lse in ((True, False) if B == 2 else (True,)):
            o.zero_()
            lse.fill_(7.0)
            st = binding.fa_forward_host(h, q.data_ptr(), k.data_ptr(), v.data_ptr(), o.data_ptr(),
                                         lse.data_ptr() if want_lse else None, B, Hq, Hkv, S, S, 128, 128, True, w.scale, stream)
            assert st == binding.FA_OK
            assert binding.fa_last_status(h) == (binding.FA_OK, 0)
            O_host = W.bf16_bits_to_f64(o.numpy().view(np.uint16))
            np.testing.assert_array_equal(O_host, O_dev)
            if want_lse:
                np.testing.assert_array_equal(lse.numpy().astype(np.float64), lse_dev)
            else:
                assert (lse.numpy() == 7.0).all()               # untouched
        rows = W.sample_rows(w, 24, seed=w.seed, heads=None)
        O_ref, lse_ref = oracle.attention(Q, K, V, causal=True, scale=w.scale, rows=rows)
        assert_parity(O_host[rows[:, 0], rows[:, 1], rows[:, 2]], lse_dev[rows[:, 0], rows[:, 1], rows[:, 2]], O_ref, lse_ref, name)
    finally:
        assert binding.fa_destroy(h) == binding.FA_OK
