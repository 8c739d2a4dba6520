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


# Every kernel has its own barrier protocol, so every one gets a wait that runs out: (name, handle flags, entry, shape).
# The shapes are tiny (a few CTAs) and the limit is 20 ms, so each case costs a few tens of milliseconds.
def _kernels():
    from paper_2609_21264_b200 import binding as b
    return [
        ("fa_fwd_pair", b.FA_FLAG_NO_STREAM_KERNEL | b.FA_FLAG_NO_PERSISTENT, "bf16", (1, 2, 2, 256, 384, 128)),
        ("fa_fwd_pipelined", b.FA_FLAG_NO_STREAM_KERNEL | b.FA_FLAG_NO_PERSISTENT | b.FA_FLAG_LEGACY_PAIR_KERNEL, "bf16", (1, 2, 2, 256, 384, 128)),
        ("fa_fwd_pipelined", b.FA_FLAG_NO_STREAM_KERNEL | b.FA_FLAG_NO_PERSISTENT, "bf16", (1, 2, 2, 256, 384, 64)),
        ("fa_fwd_stream", b.FA_FLAG_STREAM_KERNEL, "bf16", (1, 2, 1, 200, 500, 128)),
        ("fa_fwd_stream", b.FA_FLAG_STREAM_KERNEL, "bf16", (1, 2, 2, 130, 300, 192)),
        ("fa_fwd_stream_persistent", b.FA_FLAG_STREAM_KERNEL, "bf16", (8, 16, 4, 512, 640, 192)),
        ("fa_fwd_persistent", b.FA_FLAG_FORCE_PERSISTENT | b.FA_FLAG_NO_STREAM_KERNEL, "bf16", (2, 4, 2, 300, 300, 128)),
        ("fa_fwd_persistent", b.FA_FLAG_FORCE_PERSISTENT | b.FA_FLAG_NO_STREAM_KERNEL, "bf16", (2, 4, 4, 300, 300, 64)),
        ("fa_fwd_persistent", b.FA_FLAG_FORCE_PERSISTENT | b.FA_FLAG_NO_STREAM_KERNEL | b.FA_FLAG_LEGACY_PAIR_KERNEL, "bf16", (2, 4, 2, 300, 300, 128)),
        ("fa_fwd_duo", b.FA_FLAG_TWO_CTA_KERNEL, "bf16", (1, 2, 2, 256, 384, 128)),
        ("fa_fwd_duo", b.FA_FLAG_TWO_CTA_KERNEL, "bf16", (1, 4, 2, 300, 300, 192)),
        ("fa_fwd_quad", b.FA_FLAG_QUAD_KERNEL, "bf16", (1, 4, 1, 600, 700, 128)),
        ("fa_fwd_quad", b.FA_FLAG_QUAD_KERNEL, "bf16", (1, 3, 3, 300, 300, 192)),
        ("fa_fwd_fp8", b.FA_FLAG_NO_STREAM_KERNEL, "e4m3", (1, 2, 2, 256, 384, 128)),
        ("fa_fwd_fp8_stream", b.FA_FLAG_STREAM_KERNEL, "e4m3", (1, 2, 1, 200, 500, 128)),
        ("fa_fwd_mxfp8_stream", 0, "mx", (1, 2, 1, 200, 500, 128)),
    ]


@pytest.mark.parametrize("case", range(16))
def test_every_kernel_reports_a_wait_that_runs_out_and_the_handle_recovers(case):
    """The hook drops the first V tile of every CTA: the launch returns (every wait is bounded), the host reads
    FA_ERR_DEVICE_TIMEOUT with the site that gave up, and the NEXT launch through the same handle, with the hook off,
    matches the oracle: nothing the failed launch left behind (barrier state lives in the CTA; the persistent kernel's
    work-item counter is put back by fa_last_status) may leak into it."""
    import torch
    from paper_2609_21264_b200 import binding as b
    name, flags, kind, (B, Hq, Hkv, Sq, Sk, d) = _kernels()[case]
    dv = 128 if d == 192 else d
    w = W.Workload("timeout_%s_d%d" % (name, d), B, Hq, Hkv, Sq, Sk, d, dv, True, d ** -0.5, seed=70 + case)
    Q, K, V = W.make_inputs(w)
    if kind == "e4m3":
        # block-scaled codes; the oracle sees the values the codes represent
        q8, sq, qd = W.quantize_e4m3_blocks(W.bf16_bits_to_f64(Q), 128)
        k8, sk, kd = W.quantize_e4m3_blocks(W.bf16_bits_to_f64(K), 128)
        v8, sv, vd = W.quantize_e4m3_blocks(W.bf16_bits_to_f64(V), None)
    if kind == "mx":
        # e8m0 scales per 32 elements along each contraction, as scale atoms
        q8, qe, qd = W.quantize_mx_e4m3(W.bf16_bits_to_f64(Q), "cols")
        k8, ke, kd = W.quantize_mx_e4m3(W.bf16_bits_to_f64(K), "cols")
        v8, ve, vd = W.quantize_mx_e4m3(W.bf16_bits_to_f64(V), "rows")
        qa, ka, va = W.mx_scale_atoms(qe, "cols", Sq), W.mx_scale_atoms(ke, "cols", Sk), W.mx_scale_atoms(ve, "rows", Sk)
    h = b.fa_create(flags=flags | b.FA_FLAG_DEBUG_DROP_V_LOAD, wait_limit_ms=20, kv_splits=1)
    try:
        def launch():
            if kind == "bf16":
                o, lse = b.forward(h, to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V), causal=True, scale=w.scale)
            elif kind == "mx":
                o, lse = b.forward_mxfp8(h, torch.from_numpy(q8).cuda(), torch.from_numpy(k8).cuda(), torch.from_numpy(v8).cuda(),
                                         torch.from_numpy(qa).cuda(), torch.from_numpy(ka).cuda(), torch.from_numpy(va).cuda(),
                                         causal=True, scale=w.scale)
            else:
                o, lse = b.forward_fp8(h, torch.from_numpy(q8).cuda(), torch.from_numpy(k8).cuda(), torch.from_numpy(v8).cuda(),
                                       torch.from_numpy(sq).cuda(), torch.from_numpy(sk).cuda(), torch.from_numpy(sv).cuda(),
                                       causal=True, scale=w.scale)
            torch.cuda.synchronize()                  # returns: every wait is bounded
            return o, lse
        launch()
        assert b.fa_last_kernel_name(h) == name
        st, site = b.fa_last_status(h)
        assert st == b.FA_ERR_DEVICE_TIMEOUT and site != 0, (name, st, site)
        assert b.fa_last_status(h)[0] == b.FA_OK      # reading cleared it
        assert b.fa_debug_set_drop_v_load(h, False) == b.FA_OK
        o, lse = launch()
        assert b.fa_last_kernel_name(h) == name
        assert b.fa_last_status(h) == (b.FA_OK, 0)
        from parity_util import bf16_tensor_to_f64
        O, L = bf16_tensor_to_f64(o), lse.double().cpu().numpy()
        if kind == "bf16":
            O_ref, lse_ref = oracle.attention(Q, K, V, causal=True, scale=w.scale)
            assert_parity(O, L, O_ref, lse_ref, w.name)
        else:
            O_ref, lse_ref = oracle.attention(qd, kd, vd, causal=True, scale=w.scale)
            # the 8-bit path's own bound: P is rounded to e4m3 (2^-4 relative) before the second contraction
            assert np.abs(O - O_ref).max() <= 2.0 ** -4 * np.abs(vd).max() + 1e-3 and np.abs(L - lse_ref).max() <= 1e-3, w.name
    finally:
        assert b.fa_destroy(h) == b.FA_OK
