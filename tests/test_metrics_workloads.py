"""Host logic: the throughput metric's convention, work/traffic counts, input generator."""
import json
import os

import numpy as np

from paper_2609_21264_b200 import metrics as M
from paper_2609_21264_b200 import workloads as W

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def test_metric_convention_matches_the_paper_tables():
    g = json.load(open(os.path.join(GOLDEN, "paper_throughput.json")))
    for r in g["rows"]:
        f = M.flops_paper(1, r["H"], r["S"], r["S"], r["d"], r["d"])
        gflops = M.tflops_gemm(f, r["seconds"]) * 1e3
        assert abs(gflops / r["gflops"] - 1.0) < r["rel_tol"], r


def test_visible_pairs_against_enumeration():
    for Sq in range(1, 9):
        for Sk in range(1, 9):
            full = sum(1 for i in range(Sq) for j in range(Sk))
            caus = sum(1 for i in range(Sq) for j in range(Sk) if j <= i + Sk - Sq)
            assert M.visible_pairs(Sq, Sk, False) == full
            assert M.visible_pairs(Sq, Sk, True) == caus, (Sq, Sk)


def test_work_and_traffic_of_the_five_configs():
    # figures of the hot-path scope table
    exp = [(8.053e8, 8.053e8, 3.17e6), (6.872e10, 3.438e10, 42.2e6), (4.398e12, 2.1993e12, 1.078e9),
           (1.3744e12, 6.874e11, 673e6), (2.8147e14, 1.4074e14, 2.70e9)]
    for c, (fp, fa, by) in zip(W.CONFIGS, exp):
        assert abs(M.flops_paper(c.B, c.Hq, c.Sq, c.Sk, c.dqk, c.dv) / fp - 1) < 1e-3
        assert abs(M.flops_algorithmic(c.B, c.Hq, c.Sq, c.Sk, c.dqk, c.dv, c.causal) / fa - 1) < 1e-3
        assert abs(M.bytes_compulsory(c.B, c.Hq, c.Hkv, c.Sq, c.Sk, c.dqk, c.dv) / by - 1) < 2e-3


def test_roofline_picks_the_slower_side():
    t, bound = M.roofline_seconds(10**12, 10**6, 1000.0, 1000.0)
    assert bound == "tensor" and abs(t - 1e-3) < 1e-12
    t, bound = M.roofline_seconds(10**6, 10**9, 1000.0, 1000.0)
    assert bound == "hbm" and abs(t - 1e-3) < 1e-12


def test_bf16_rounding_is_nearest_even():
    import torch
    x = np.random.default_rng(0).standard_normal(100000).astype(np.float32) * 3
    x[:4] = [1.00390625, 1.01171875, -1.00390625, 0.0]   # exact ties: to even
    bits = W.f32_to_bf16_bits(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(bits, ref)
    back = W.bf16_bits_to_f64(bits)
    np.testing.assert_array_equal(back, torch.from_numpy(x).to(torch.bfloat16).double().numpy())


def test_generator_is_seeded_and_shaped():
    w = W.config(0)
    Q, K, V = W.make_inputs(w)
    Q2, K2, V2 = W.make_inputs(w)
    assert Q.dtype == np.uint16 and Q.shape == (1, 12, 512, 64) and V.shape == (1, 12, 512, 64)
    np.testing.assert_array_equal(Q, Q2)
    assert not np.array_equal(Q, K) and not np.array_equal(K, V)
    q = W.bf16_bits_to_f64(Q)
    assert abs(q.mean()) < 0.01 and abs(q.std() - 1.0) < 0.01
    w3 = W.config(2).with_(B=1, Hq=2, Hkv=2, Sq=256, Sk=256)
    _, K3, _ = W.make_inputs(w3)
    assert abs(W.bf16_bits_to_f64(K3).std() - 2.0) < 0.02      # K scaled by 2
    assert W.make_inputs(w.with_(seed=7))[0].tobytes() != Q.tobytes()


def test_sample_rows_are_in_range():
    w = W.config(4)
    rows = W.sample_rows(w, 32, seed=1, heads=[0, 31])
    assert rows.shape[1] == 3 and (rows[:, 2] < w.Sq).all() and (rows[:, 1] < w.Hq).all()
    assert {0, 127, 128, w.Sq - 1} <= set(rows[:, 2].tolist())


def _decode_e4m3(codes):
    """e4m3 ("fn": no infinities, 0x7f/0xff are NaN) written out: 1 sign, 4 exponent (bias 7), 3 mantissa bits."""
    c = codes.astype(np.int64)
    s, e, m = c >> 7, (c >> 3) & 15, c & 7
    mag = np.where(e == 0, m * 2.0 ** -9, (1.0 + m / 8.0) * 2.0 ** (e - 7.0))
    return np.where(s == 1, -mag, mag)


def test_block_quantiser_of_the_8_bit_path():
    """What the 8-bit tests hand to the oracle (codes x scales) is what the codes mean under the
    format's definition, the scales are amax / 448 per block, and every value is rounded to a
    nearest representable one."""
    from paper_2609_21264_b200 import workloads as W
    rng = np.random.default_rng(5)
    x = rng.standard_normal((2, 3, 300, 64)) * rng.uniform(0.01, 30.0, size=(2, 3, 300, 1))
    x[0, 0, :128] = 0.0                                         # an all-zero block keeps scale 1
    for block_rows in (128, None):
        codes, scales, deq = W.quantize_e4m3_blocks(x, block_rows)
        assert codes.dtype == np.uint8 and codes.shape == x.shape and scales.dtype == np.float32
        assert not np.isin(codes, (0x7f, 0xff)).any()           # no NaN codes
        if block_rows:
            per_row = np.repeat(scales.astype(np.float64), block_rows, axis=2)[:, :, :300, None]
            amax = np.stack([np.abs(x[:, :, i:i + block_rows]).max(axis=(2, 3)) for i in range(0, 300, block_rows)], axis=2)
        else:
            per_row = scales.astype(np.float64)[:, :, None, None]
            amax = np.abs(x).max(axis=(2, 3))
        assert np.array_equal(deq, _decode_e4m3(codes) * per_row)
        want = np.where(amax > 0, amax / 448.0, 1.0).astype(np.float32)
        assert np.array_equal(scales, want)
        # nearest: the error is at most half a step of the format at that magnitude (3 mantissa bits; the
        # fp32 scale and quotient add a few parts in 1e7)
        y = x / per_row
        step = np.where(np.abs(y) < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y), 2.0 ** -6))) - 3))
        assert (np.abs(_decode_e4m3(codes) - y) <= 0.5 * step * (1 + 1e-6) + 1e-9).all()
        assert (np.abs(_decode_e4m3(codes)) <= 448.0).all()


def test_mx_quantiser_and_scale_atoms():
    """quantize_mx_e4m3: power-of-two scales per 32 elements, the smallest that avoids saturation, nearest-even codes;
    mx_scale_atoms: byte (r % 32) * 16 + (r / 32) * 4 + kb of a tile's 512-byte atom, padding 127."""
    rng = np.random.default_rng(12)
    x = rng.standard_normal((2, 3, 300, 64)) * np.exp2(rng.integers(-12, 13, size=(2, 3, 300, 1)).astype(np.float64))
    x[0, 0, 5, :32] = 0.0                                        # an all-zero block keeps the scale 2^0
    for along in ("cols", "rows"):
        codes, exps, deq = W.quantize_mx_e4m3(x, along)
        assert codes.dtype == np.uint8 and exps.dtype == np.uint8 and codes.shape == x.shape
        assert not np.isin(codes, (0x7f, 0xff)).any() and exps.max() < 255
        if along == "cols":
            assert exps.shape == (2, 3, 300, 2)
            per_elem = np.repeat(np.exp2(exps.astype(np.float64) - 127.0), 32, axis=3)
            amax = np.abs(x).reshape(2, 3, 300, 2, 32).max(axis=4)
            assert exps[0, 0, 5, 0] == 127
        else:
            assert exps.shape == (2, 3, 10, 64)
            per_elem = np.repeat(np.exp2(exps.astype(np.float64) - 127.0), 32, axis=2)[:, :, :300]
            xp = np.concatenate([x, np.zeros((2, 3, 20, 64))], axis=2)
            amax = np.abs(xp).reshape(2, 3, 10, 32, 64).max(axis=3)
        assert np.array_equal(deq, _decode_e4m3(codes) * per_elem)
        scale = np.exp2(exps.astype(np.float64) - 127.0)
        nz = amax > 0
        assert (amax[nz] / scale[nz] <= 448.0).all() and (amax[nz] / scale[nz] > 224.0).all()     # the smallest such power of two
        y = x / per_elem
        step = np.where(np.abs(y) < 2.0 ** -6, 2.0 ** -9, 2.0 ** (np.floor(np.log2(np.maximum(np.abs(y), 2.0 ** -6))) - 3))
        assert (np.abs(_decode_e4m3(codes) - y) <= 0.5 * step * (1 + 1e-6) + 1e-9).all()
        atoms = W.mx_scale_atoms(exps, along, 300)
        assert atoms.shape == (2, 3, 3, 512) and atoms.dtype == np.uint8
        for _ in range(200):
            b, h, t, r, kb = rng.integers(2), rng.integers(3), rng.integers(3), rng.integers(128), rng.integers(4)
            byte = atoms[b, h, t, (r % 32) * 16 + (r // 32) * 4 + kb]
            if along == "cols":
                row = 128 * t + r
                want = exps[b, h, row, kb] if (row < 300 and kb < 2) else 127
            else:
                blk = 4 * t + kb
                want = exps[b, h, blk, r] if (blk < 10 and r < 64) else 127
            assert byte == want
