"""Seeded random shapes through the default handle (the library picks kernel, tiling and split count)
against the oracle: every selection path has to agree with the definition, whatever it chooses."""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, run_gpu

pytestmark = pytest.mark.gpu


def _cases():
    rng = np.random.default_rng(20261125)
    out = []
    for i in range(36):
        d = int(rng.choice([64, 128, 192]))
        hkv = int(rng.choice([1, 2, 3, 4]))
        gqa = int(rng.choice([1, 1, 2, 4]))
        kind = i % 4
        if kind == 0:      # short self-attention, several heads
            sq = sk = int(rng.integers(1, 700))
            b = int(rng.integers(1, 4))
        elif kind == 1:    # decode / cross attention: few queries, many keys
            sq, sk, b = int(rng.integers(1, 140)), int(rng.integers(1500, 6000)), 1
        elif kind == 2:    # more queries than keys
            sq, sk, b = int(rng.integers(200, 900)), int(rng.integers(1, 400)), 1
        else:              # longer sequences, one K/V head
            sq = sk = int(rng.integers(900, 2600))
            b, hkv = 1, 1
        causal = bool(rng.integers(0, 2))
        out.append(W.Workload("rand%02d_b%d_h%dx%d_%dx%d_d%d_%s" % (i, b, hkv, gqa, sq, sk, d, "c" if causal else "f"),
                              B=b, Hq=hkv * gqa, Hkv=hkv, Sq=sq, Sk=sk, dqk=d, dv=128 if d == 192 else d,
                              causal=causal, scale=d ** -0.5, seed=7000 + i))
    return out


CASES = _cases()


@pytest.fixture(scope="module")
def handle():
    from paper_2609_21264_b200 import binding
    h = binding.fa_create()
    yield h
    binding.fa_destroy(h)


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_random_shape_matches_oracle(handle, w):
    Q, K, V = W.make_inputs(w)
    heads = sorted({0, w.Hq - 1})
    if w.Sq * w.Sk > 1_500_000:      # keep the oracle's share of the run short: sampled rows
        rows = W.sample_rows(w, 96, seed=w.seed, heads=heads)
        O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale, rows=rows)
        O, lse = run_gpu(handle, w, Q, K, V)
        assert np.isfinite(O).all()
        assert_parity(O[rows[:, 0], rows[:, 1], rows[:, 2]], lse[rows[:, 0], rows[:, 1], rows[:, 2]], O_ref, lse_ref, w.name)
    else:
        O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
        O, lse = run_gpu(handle, w, Q, K, V)
        assert_parity(O, lse, O_ref, lse_ref, w.name)


def _decode_cases():
    """Few queries per sequence with grouped heads: the shapes whose heads share a query tile."""
    rng = np.random.default_rng(20261126)
    out = []
    for i in range(24):
        d = int(rng.choice([64, 128, 128, 192]))
        hkv = int(rng.integers(1, 4))
        gqa = int(rng.choice([2, 3, 4, 6, 8, 16]))
        sq = int(rng.choice([1, 1, 2, 3, 5, 8, 16, 17, 31, 32, 33, 64]))
        sk = int(rng.integers(sq, 5000))
        b = int(rng.integers(1, 4))
        causal = bool(rng.integers(0, 2))
        out.append(W.Workload("dec%02d_b%d_h%dx%d_%dx%d_d%d_%s" % (i, b, hkv, gqa, sq, sk, d, "c" if causal else "f"),
                              B=b, Hq=hkv * gqa, Hkv=hkv, Sq=sq, Sk=sk, dqk=d, dv=128 if d == 192 else d,
                              causal=causal, scale=d ** -0.5, seed=7100 + i))
    return out


DECODE_CASES = _decode_cases()


@pytest.mark.parametrize("w", DECODE_CASES, ids=[w.name for w in DECODE_CASES])
def test_random_decode_shape_matches_oracle(handle, w):
    import torch
    from paper_2609_21264_b200 import binding
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    O, lse = run_gpu(handle, w, Q, K, V)
    plan = binding.fa_plan(torch.cuda.get_device_properties(0).multi_processor_count, w.B, w.Hq, w.Hkv, w.Sq, w.Sk,
                           w.dqk, w.dv, w.causal)
    assert binding.fa_last_kernel_name(handle) == plan["kernel"] and binding.fa_last_kv_splits(handle) == plan["kv_splits"]
    assert_parity(O, lse, O_ref, lse_ref, w.name)


@pytest.mark.parametrize("w", [w for w in DECODE_CASES if w.dqk in (64, 128)],
                         ids=[w.name for w in DECODE_CASES if w.dqk in (64, 128)])
def test_random_decode_shape_e4m3_matches_oracle_on_represented_tensors(handle, w):
    import torch
    from paper_2609_21264_b200 import binding
    from parity_util import bf16_tensor_to_f64, LSE_MAX_ABS
    Q, K, V = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
    q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
    k8, sk, Kd = W.quantize_e4m3_blocks(K, 128)
    v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
    O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=w.causal, scale=w.scale)
    dev = lambda a: torch.from_numpy(a).cuda()
    o, lse = binding.forward_fp8(handle, dev(q8), dev(k8), dev(v8), dev(sq), dev(sk), dev(sv), causal=w.causal, scale=w.scale)
    torch.cuda.synchronize()
    st, detail = binding.fa_last_status(handle)
    assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)
    O, lse = bf16_tensor_to_f64(o), lse.double().cpu().numpy()
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(lse), np.isneginf(lse_ref))
    assert np.abs(lse[fin] - lse_ref[fin]).max() <= LSE_MAX_ABS
    err = np.abs(O - O_ref)
    vmax = np.abs(Vd).max(axis=(2, 3))
    bound = 2.0 ** -4 * np.repeat(vmax, w.Hq // w.Hkv, axis=1)[:, :, None, None] + 2.0 ** -8 * np.abs(O_ref) + 1e-3
    assert (err <= bound).all(), (w.name, float(err.max()), float((err / bound).max()))
    assert err.mean() <= 1e-2, (w.name, float(err.mean()))
