"""The bounded device-side waits: a wait that can never be satisfied runs into its limit, the kernel
returns, the host reads FA_ERR_DEVICE_TIMEOUT, and the context stays usable.

The failure is made on purpose in the gentlest way there is: the load warp leaves out one TMA
load (a test hook of the library), so the mbarrier the MMA threads wait on is never armed.
Nothing faults, traps or spins without bound.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, run_gpu, to_torch_bf16

pytestmark = pytest.mark.gpu


def test_wait_limit_reports_timeout_and_context_survives():
    import torch
    from paper_2609_21264_b200 import binding as b
    w = W.Workload("tiny", 1, 1, 1, 256, 256, 128, 128, False, 128 ** -0.5, seed=5)
    Q, K, V = W.make_inputs(w)
    q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
    h = b.fa_create(flags=b.FA_FLAG_DEBUG_DROP_V_LOAD, wait_limit_ms=20, kv_splits=1)
    try:
        o, lse = b.forward(h, q, k, v, causal=False, scale=w.scale)
        torch.cuda.synchronize()                      # returns: every wait is bounded
        st, site = b.fa_last_status(h)
        assert st == b.FA_ERR_DEVICE_TIMEOUT
        assert site != 0                              # the role and barrier that gave up
        assert b.fa_last_status(h)[0] == b.FA_OK      # reading cleared it
    finally:
        assert b.fa_destroy(h) == b.FA_OK
    # the same context keeps working
    h2 = b.fa_create()
    try:
        O_ref, lse_ref = oracle.attention(Q, K, V, causal=False, scale=w.scale)
        O, lse2 = run_gpu(h2, w, Q, K, V)
        assert_parity(O, lse2, O_ref, lse_ref, "after timeout")
    finally:
        b.fa_destroy(h2)
