"""The paper's numerical-stability protocol (Section 5.5) as a regression test against the fp64 oracle.

GPT-2-Small attention shape, inputs N(0, sigma^2) with sigma from 0.25 to 4: mean absolute error
and per-head Pearson correlation.  The paper's kernel keeps scores and softmax state in bf16 and
its printed curve is the envelope here: a kernel with fp32 state must stay below it.  The paper
does not say whether its run was causal; both modes are checked.
"""
import json
import os

import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import run_gpu

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "paper_sigma_sweep.json")


@pytest.fixture(scope="module")
def handle():
    from paper_2609_21264_b200 import binding
    h = binding.fa_create()
    yield h
    binding.fa_destroy(h)


@pytest.mark.parametrize("causal", [True, False])
def test_sigma_sweep_stays_below_the_papers_error_curve(handle, causal):
    g = json.load(open(GOLDEN))
    H, d, S = g["shape"]["H"], g["shape"]["d"], g["shape"]["S"]
    report = []
    for sigma, mae_paper, rho_paper in zip(g["sigma"], g["mae_x1e-2"], g["pearson"]):
        w = W.Workload("sweep", 1, H, H, S, S, d, d, causal, d ** -0.5, sigma=sigma, seed=1234)
        Q, K, V = W.make_inputs(w)
        O_ref, lse_ref = oracle.attention(Q, K, V, causal=causal, scale=w.scale)
        O, lse = run_gpu(handle, w, Q, K, V)
        mae = float(np.abs(O - O_ref).mean())
        rho = min(float(np.corrcoef(O[0, h].ravel(), O_ref[0, h].ravel())[0, 1]) for h in range(H))
        report.append((sigma, mae, mae_paper * 1e-2, rho, rho_paper))
        assert np.isfinite(O).all() and np.isfinite(lse).all()
        assert mae <= mae_paper * 1e-2, (sigma, mae, mae_paper * 1e-2)       # below the bf16-state kernel
        assert rho >= 0.9999, (sigma, rho)                                   # the paper reports >= 0.9987
        # what bf16 output rounding alone allows: |O| ~ sigma, relative half-ulp 2^-9
        assert mae <= 2.0 ** -9 * sigma + 1e-5, (sigma, mae)
        assert np.abs(lse - lse_ref).max() <= 1e-3 * max(1.0, sigma ** 2), (sigma,)
    for row in report:
        print("sigma %.2f  MAE %.2e (paper %.2e)  min Pearson %.6f (paper %.4f)" % row)


@pytest.mark.parametrize("d", [64, 128], ids=["d64_the_papers_shape", "d128"])
def test_sigma_sweep_of_the_block_scaled_e4m3_path(d):
    """The same protocol for the 8-bit variant: Q, K (one scale per 128-row block) and V (one per
    head) quantised to e4m3 from the same N(0, sigma^2) inputs.

    Two errors per sigma.  Against the oracle on the tensors the codes REPRESENT: what the kernel
    adds (P rounded to e4m3 before the second contraction, fp32 state, bf16 output).  Against the
    oracle on the ORIGINAL inputs: what a user of the 8-bit path sees, dominated by the
    quantisation of the inputs (relative 2^-4 per element; the scores' error grows with sigma^2
    and the softmax sharpens, so this error is largest at the top of the sweep).  The kernel's own
    error is held against the paper's curve for its bf16-state kernel; the end-to-end error is
    reported and held to regression bounds (it is a property of the format, not of the kernel).
    """
    import torch
    from paper_2609_21264_b200 import binding
    g = json.load(open(GOLDEN))
    H, S = g["shape"]["H"], g["shape"]["S"]
    h = binding.fa_create()
    report = []
    try:
        for sigma, mae_paper in zip(g["sigma"], g["mae_x1e-2"]):
            w = W.Workload("sweep8", 1, H, H, S, S, d, d, True, d ** -0.5, sigma=sigma, seed=4321)
            Q, K, V = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
            q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
            k8, sk, Kd = W.quantize_e4m3_blocks(K, 128)
            v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
            O_rep, lse_rep = oracle.attention(Qd, Kd, Vd, causal=True, scale=w.scale)
            O_org, _ = oracle.attention(Q, K, V, causal=True, scale=w.scale)
            dev = lambda a: torch.from_numpy(a).cuda()
            o, lse = binding.forward_fp8(h, dev(q8), dev(k8), dev(v8), dev(sq), dev(sk), dev(sv), causal=True, scale=w.scale)
            torch.cuda.synchronize()
            assert binding.fa_last_status(h)[0] == binding.FA_OK
            O = o.double().cpu().numpy()
            lse = lse.double().cpu().numpy()
            mae_k = float(np.abs(O - O_rep).mean())
            mae_e = float(np.abs(O - O_org).mean())
            rho_k = min(float(np.corrcoef(O[0, i].ravel(), O_rep[0, i].ravel())[0, 1]) for i in range(H))
            rho_e = min(float(np.corrcoef(O[0, i].ravel(), O_org[0, i].ravel())[0, 1]) for i in range(H))
            report.append((sigma, mae_k, mae_paper * 1e-2, rho_k, mae_e, rho_e))
            assert np.isfinite(O).all() and np.isfinite(lse).all()
            assert np.abs(lse - lse_rep).max() <= 1e-3 * max(1.0, sigma ** 2), (sigma,)
            # measured 1.8e-4 .. 2.4e-2 over the sweep: below the paper's curve from sigma = 1 on, within a
            # factor two of it below (there that curve sits at the bf16 output rounding and the three
            # mantissa bits of P show)
            assert mae_k <= mae_paper * 1e-2 * (2.0 if sigma < 1.0 else 1.0), (sigma, mae_k)
            assert rho_k >= 0.9995, (sigma, rho_k)
            # measured 2.9e-4 .. 0.29 and Pearson 0.9994 .. 0.986: regression bounds with some margin
            assert mae_e <= 0.09 * sigma, (sigma, mae_e)
            assert rho_e >= 0.98, (sigma, rho_e)
    finally:
        binding.fa_destroy(h)
        for row in report:
            print("sigma %.2f  kernel MAE %.2e (paper's bf16 curve %.2e) min Pearson %.6f | with input quantisation MAE %.2e Pearson %.6f" % row)


@pytest.mark.parametrize("d", [64, 128], ids=["d64_the_papers_shape", "d128"])
def test_sigma_sweep_of_the_mx_path(d):
    """The same protocol for the MX form (fa_forward_mxfp8): e8m0 scales per 32 elements along each contraction.
    Kernel error against the oracle on the represented tensors, end-to-end error against the oracle on the original
    inputs.  On these i.i.d. inputs every block has the same magnitude, so the figures equal those of one scale per
    128-row block to two digits (measured, both tables are in the design document); what scales every 32 elements
    buy shows on inputs whose rows and columns differ in magnitude (tests/test_gpu_mxfp8.py)."""
    import torch
    from paper_2609_21264_b200 import binding
    g = json.load(open(GOLDEN))
    H, S = g["shape"]["H"], g["shape"]["S"]
    h = binding.fa_create()
    report = []
    try:
        for sigma, mae_paper in zip(g["sigma"], g["mae_x1e-2"]):
            w = W.Workload("sweep_mx", 1, H, H, S, S, d, d, True, d ** -0.5, sigma=sigma, seed=4321)
            Q, K, V = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
            q8, qe, Qd = W.quantize_mx_e4m3(Q, "cols")
            k8, ke, Kd = W.quantize_mx_e4m3(K, "cols")
            v8, ve, Vd = W.quantize_mx_e4m3(V, "rows")
            O_rep, lse_rep = oracle.attention(Qd, Kd, Vd, causal=True, scale=w.scale)
            O_org, _ = oracle.attention(Q, K, V, causal=True, scale=w.scale)
            dev = lambda a: torch.from_numpy(a).cuda()
            o, lse = binding.forward_mxfp8(h, dev(q8), dev(k8), dev(v8), dev(W.mx_scale_atoms(qe, "cols", S)),
                                           dev(W.mx_scale_atoms(ke, "cols", S)), dev(W.mx_scale_atoms(ve, "rows", S)),
                                           causal=True, scale=w.scale)
            torch.cuda.synchronize()
            assert binding.fa_last_status(h)[0] == binding.FA_OK
            O = o.double().cpu().numpy()
            lse = lse.double().cpu().numpy()
            mae_k = float(np.abs(O - O_rep).mean())
            mae_e = float(np.abs(O - O_org).mean())
            rho_k = min(float(np.corrcoef(O[0, i].ravel(), O_rep[0, i].ravel())[0, 1]) for i in range(H))
            rho_e = min(float(np.corrcoef(O[0, i].ravel(), O_org[0, i].ravel())[0, 1]) for i in range(H))
            report.append((sigma, mae_k, mae_paper * 1e-2, rho_k, mae_e, rho_e))
            assert np.isfinite(O).all() and np.isfinite(lse).all()
            assert np.abs(lse - lse_rep).max() <= 1e-3 * max(1.0, sigma ** 2), (sigma,)
            # the kernel's own error is that of the e4m3 path (the same rounding of P): same bounds
            assert mae_k <= mae_paper * 1e-2 * (2.0 if sigma < 1.0 else 1.0), (sigma, mae_k)
            assert rho_k >= 0.9995, (sigma, rho_k)
            assert mae_e <= 0.09 * sigma, (sigma, mae_e)
            assert rho_e >= 0.98, (sigma, rho_e)
    finally:
        binding.fa_destroy(h)
        for row in report:
            print("sigma %.2f  kernel MAE %.2e (paper's bf16 curve %.2e) min Pearson %.6f | with input quantisation MAE %.2e Pearson %.6f" % row)
