"""MX form of the 8-bit path (fa_forward_mxfp8): e4m3 values with one e8m0 scale per 32 elements along each
contraction, applied inside tcgen05.mma kind::mxf8f6f4 with block scaling, against the oracle.

As for fa_forward_fp8 the oracle gets the tensors the inputs REPRESENT (codes x 2^(e - 127), exact in fp64), so the
comparison isolates what the kernel adds: fp32 accumulation, probabilities rounded to e4m3 (scale 1) before the second
contraction, bf16 output.  lse only depends on the first contraction and the fp32 softmax state (bound 1e-3, as for
bf16): with scales that differ from row to row and from block to block it pins the layout of the Q and K scale atoms.
O: |O - O_ref| <= 2^-4 max|V| per element in the worst case (one dominant key), far less on spread-out rows.  The
layout of the V scale atom (per column and block of 32 keys) is pinned by the K = 0 case, where every probability is
exactly 1, and by moving powers of two between codes and scales, which must not change the result.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import bf16_tensor_to_f64, LSE_MAX_ABS

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handle():
    from paper_2609_21264_b200 import binding
    h = binding.fa_create()
    yield h
    binding.fa_destroy(h)


def _run(handle, w, q8, k8, v8, qa, ka, va):
    import torch
    from paper_2609_21264_b200 import binding
    dev = lambda a: torch.from_numpy(a).cuda()
    o, lse = binding.forward_mxfp8(handle, dev(q8), dev(k8), dev(v8), dev(qa), dev(ka), dev(va), causal=w.causal, scale=w.scale)
    torch.cuda.synchronize()
    st, detail = binding.fa_last_status(handle)
    assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)
    assert binding.fa_last_kernel_name(handle) == "fa_fwd_mxfp8_stream"
    return bf16_tensor_to_f64(o), lse.double().cpu().numpy()


def _wl(name, B, Hq, Hkv, Sq, Sk, causal, seed, d=128):
    return W.Workload(name, B=B, Hq=Hq, Hkv=Hkv, Sq=Sq, Sk=Sk, dqk=d, dv=d, causal=causal, scale=d ** -0.5, seed=seed)


def _inputs(w, spread=True):
    """N(0,1) values; with `spread`, rows of Q and K and columns of V additionally differ by powers of two (up to 2^3
    either way for Q and V, 2^2 for K), which is what scales per 32 elements are for and what a single scale per
    128-row block could not hold in e4m3's range."""
    rng = np.random.default_rng(w.seed)
    Q = rng.standard_normal((w.B, w.Hq, w.Sq, w.dqk))
    K = rng.standard_normal((w.B, w.Hkv, w.Sk, w.dqk))
    V = rng.standard_normal((w.B, w.Hkv, w.Sk, w.dv))
    if spread:
        Q = Q * np.exp2(rng.integers(-3, 4, size=(w.B, w.Hq, w.Sq, 1)))
        K = K * np.exp2(rng.integers(-2, 3, size=(w.B, w.Hkv, w.Sk, 1))) * 0.5
        V = V * np.exp2(rng.integers(-3, 4, size=(w.B, w.Hkv, 1, w.dv)))
    return Q, K, V


def _quantise(w, Q, K, V):
    q8, qe, Qd = W.quantize_mx_e4m3(Q, "cols")
    k8, ke, Kd = W.quantize_mx_e4m3(K, "cols")
    v8, ve, Vd = W.quantize_mx_e4m3(V, "rows")
    return (q8, k8, v8, W.mx_scale_atoms(qe, "cols", w.Sq), W.mx_scale_atoms(ke, "cols", w.Sk), W.mx_scale_atoms(ve, "rows", w.Sk)), (Qd, Kd, Vd)


def _check(w, O, lse, O_ref, lse_ref, Vd, mean_bound):
    assert np.isfinite(O).all()
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(lse), np.isneginf(lse_ref))
    assert np.abs(lse[fin] - lse_ref[fin]).max() <= LSE_MAX_ABS
    err = np.abs(O - O_ref)
    vmax = np.abs(Vd).max(axis=2)                                   # [B, Hkv, dv]: the bound holds per column
    bound = 2.0 ** -4 * np.repeat(vmax, w.Hq // w.Hkv, axis=1)[:, :, None, :] + 2.0 ** -8 * np.abs(O_ref) + 1e-3
    assert (err <= bound).all(), (w.name, float(err.max()), float((err / bound).max()))
    assert err.mean() <= mean_bound, (w.name, float(err.mean()))


CASES = [
    _wl("mx_one_tile", 1, 1, 1, 128, 128, False, 2201),
    _wl("mx_gqa_causal_ragged", 2, 8, 2, 333, 333, True, 2202),
    _wl("mx_mha_full_sq_ne_sk", 1, 4, 4, 200, 457, False, 2203),
    _wl("mx_causal_more_q_than_k", 1, 3, 3, 400, 140, True, 2204),
    _wl("mx_llama_like_s1024", 1, 8, 2, 1024, 1024, True, 2205),
    _wl("mx_one_tile_many_keys", 1, 2, 1, 100, 2100, False, 2206),          # split-KV
    _wl("mx_short_q_causal_long_k", 2, 4, 2, 130, 1500, True, 2207),
    _wl("mx_grouped_single_query", 1, 12, 2, 1, 2500, False, 2208),         # decode: one head per tile on this path
    _wl("mx_d64_gqa_causal_ragged", 2, 8, 2, 333, 333, True, 2210, d=64),
    _wl("mx_d64_gpt2_like_s1024", 1, 12, 12, 1024, 1024, True, 2211, d=64),
    _wl("mx_d64_one_tile_many_keys", 1, 2, 1, 100, 2100, False, 2212, d=64),
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_mx_matches_oracle_on_represented_tensors(handle, w):
    Q, K, V = _inputs(w)
    dev_in, (Qd, Kd, Vd) = _quantise(w, Q, K, V)
    O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=w.causal, scale=w.scale)
    O, lse = _run(handle, w, *dev_in)
    # columns of V reach 2^3 here, and the rows are sharp (scores up to a few tens): the mean error scales with both
    _check(w, O, lse, O_ref, lse_ref, Vd, mean_bound=4e-2)


def test_mx_unit_spread_inputs_meet_the_e4m3_paths_mean_bound(handle):
    """Plain N(0,1) inputs: the same accuracy class as fa_forward_fp8 (mean error 1e-2)."""
    w = _wl("mx_plain", 1, 4, 2, 512, 512, True, 2220)
    Q, K, V = _inputs(w, spread=False)
    dev_in, (Qd, Kd, Vd) = _quantise(w, Q, K, V)
    O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=True, scale=w.scale)
    O, lse = _run(handle, w, *dev_in)
    _check(w, O, lse, O_ref, lse_ref, Vd, mean_bound=1e-2)


@pytest.mark.parametrize("d", [128, 64])
def test_mx_uniform_scores_give_exact_column_means(handle, d):
    """K = 0 makes every visible probability exactly 1: O is the running mean of the represented V, to bf16 rounding.
    V's columns and 32-key blocks all carry different scales, so a misplaced byte of the V atom shows at once."""
    w = _wl("mx_uniform_d%d" % d, 1, 2, 1, 300, 300, True, 2230 + d, d=d)
    rng = np.random.default_rng(w.seed)
    Q = rng.standard_normal((1, 2, 300, d))
    # every (block of 32 keys, column) has a magnitude of its own
    V = rng.standard_normal((1, 1, 300, d)) * np.repeat(np.exp2(rng.integers(-6, 7, size=(1, 1, 10, d)).astype(np.float64)), 32, axis=2)[:, :, :300]
    q8, qe, _ = W.quantize_mx_e4m3(Q, "cols")
    v8, ve, Vd = W.quantize_mx_e4m3(V, "rows")
    assert len(np.unique(ve)) >= 8                                   # many different scales
    k8 = np.zeros((1, 1, 300, d), dtype=np.uint8)
    ka = np.full((1, 1, 3, 512), 127, dtype=np.uint8)
    O, lse = _run(handle, w, q8, k8, v8, W.mx_scale_atoms(qe, "cols", 300), ka, W.mx_scale_atoms(ve, "rows", 300))
    ref = np.cumsum(Vd[0, 0], axis=0) / np.arange(1, 301)[:, None]
    for h in range(2):
        assert (np.abs(O[0, h] - ref) <= 2.0 ** -8 * np.abs(ref) + 2.0 ** -20 * np.abs(Vd[0, 0]).max(axis=0)[None, :] + 1e-7).all()
        # (a quarter of the exponentials come from the FMA-pipe polynomial, relative error 7.5e-5: 2^0 is 0.999925 there)
        assert np.abs(lse[0, h] - np.log(np.arange(1, 301))).max() <= 5e-5


def test_mx_powers_of_two_move_between_codes_and_scales(handle):
    """Halving the codes of a block (exact for normal e4m3 numbers) and adding one to its exponent byte leaves the
    represented tensor unchanged, hence the result: for blocks of Q, of K (per row and 32 columns) and of V (per
    column and 32 keys)."""
    w = _wl("mx_resplit", 1, 2, 2, 260, 260, False, 2240)
    Q, K, V = _inputs(w)
    (q8, k8, v8, qa, ka, va), _ = _quantise(w, Q, K, V)
    O1, lse1 = _run(handle, w, q8, k8, v8, qa, ka, va)
    rng = np.random.default_rng(1)

    def resplit(codes, atoms, along):
        c, a = codes.copy(), atoms.copy()
        moved = 0
        B, H, S, d = c.shape
        for _ in range(400):
            b, h = rng.integers(B), rng.integers(H)
            if along == "cols":
                r, kb = rng.integers(S), rng.integers(d // 32)
                blk = (b, h, r, slice(32 * kb, 32 * kb + 32))
                t, rr = divmod(r, 128)
            else:
                col, kblk = rng.integers(d), rng.integers((S + 31) // 32)
                blk = (b, h, slice(32 * kblk, min(32 * kblk + 32, S)), col)
                t, kb = divmod(kblk, 4)
                rr = col
            sub = c[blk]
            if not (((sub >> 3) & 15) >= 2).all():
                continue                                            # a subnormal or zero code cannot be halved exactly
            c[blk] = sub - 8
            a[b, h, t, (rr % 32) * 16 + (rr // 32) * 4 + kb] += 1
            moved += 1
        assert moved >= 20
        return c, a

    q8b, qab = resplit(q8, qa, "cols")
    k8b, kab = resplit(k8, ka, "cols")
    v8b, vab = resplit(v8, va, "rows")
    O2, lse2 = _run(handle, w, q8b, k8b, v8b, qab, kab, vab)
    np.testing.assert_array_equal(lse1, lse2)
    np.testing.assert_array_equal(O1, O2)


def test_mx_argument_errors(handle):
    import torch
    from paper_2609_21264_b200 import binding
    z = torch.zeros((1, 1, 128, 128), dtype=torch.uint8, device="cuda")
    a = torch.full((1, 1, 1, 512), 127, dtype=torch.uint8, device="cuda")
    o = torch.zeros((1, 1, 128, 128), dtype=torch.bfloat16, device="cuda")
    args = (1, 1, 1, 128, 128)
    assert binding.fa_forward_mxfp8(handle, z.data_ptr(), z.data_ptr(), z.data_ptr(), None, a.data_ptr(), a.data_ptr(), o.data_ptr(), None,
                                    *args, 128, False, 0.0) == binding.FA_ERR_INVALID_ARG
    assert binding.fa_forward_mxfp8(handle, z.data_ptr(), z.data_ptr(), z.data_ptr(), a.data_ptr() + 4, a.data_ptr(), a.data_ptr(), o.data_ptr(),
                                    None, *args, 128, False, 0.0) == binding.FA_ERR_INVALID_ARG
    z192 = torch.zeros((1, 1, 128, 192), dtype=torch.uint8, device="cuda")
    assert binding.fa_forward_mxfp8(handle, z192.data_ptr(), z192.data_ptr(), z192.data_ptr(), a.data_ptr(), a.data_ptr(), a.data_ptr(),
                                    o.data_ptr(), None, *args, 192, False, 0.0) == binding.FA_ERR_UNSUPPORTED
    assert binding.fa_forward_mxfp8(handle, z.data_ptr(), z.data_ptr(), z.data_ptr(), a.data_ptr(), a.data_ptr(), a.data_ptr(), o.data_ptr(),
                                    None, *args, 128, False, 0.0) == binding.FA_OK
    torch.cuda.synchronize()
    assert binding.fa_last_status(handle) == (binding.FA_OK, 0)


def test_fuzz_mx_and_8bit_192(handle):
    """Seeded random problems through the two newest 8-bit forms (the MX entry at head sizes 64 and 128, and
    fa_forward_fp8 at 192/128), whatever split count the library plans for them, each against the oracle on the
    represented tensors."""
    import torch
    from paper_2609_21264_b200 import binding
    rng = np.random.default_rng(20261205)
    dev = lambda a: torch.from_numpy(a).cuda()
    splits_seen = set()
    for it in range(48):
        mx = bool(it % 2)
        d = int(rng.choice([64, 128])) if mx else 192
        dv = 128 if d == 192 else d
        hkv, gqa, B = int(rng.integers(1, 4)), int(rng.choice([1, 2, 4, 6])), int(rng.integers(1, 3))
        causal = bool(rng.integers(0, 2))
        shape = int(rng.integers(0, 4))
        if shape == 0:
            sq, sk = int(rng.integers(1, 65)), int(rng.integers(1, 5000))        # decode-like
        elif shape == 1:
            sq = sk = int(rng.integers(1, 900))
        elif shape == 2:
            sq, sk = int(rng.integers(100, 700)), int(rng.integers(1, 300))      # more queries than keys
        else:
            sq, sk = int(rng.integers(65, 300)), int(rng.integers(1000, 4000))
        name = "case%d %s b%d h%dx%d %dx%d d%d %s" % (it, "mx" if mx else "e4m3", B, hkv, gqa, sq, sk, d, "causal" if causal else "full")
        w = W.Workload(name, B=B, Hq=hkv * gqa, Hkv=hkv, Sq=sq, Sk=sk, dqk=d, dv=dv, causal=causal, scale=d ** -0.5, seed=31000 + it)
        Q = rng.standard_normal((B, w.Hq, sq, d)); K = rng.standard_normal((B, hkv, sk, d)); V = rng.standard_normal((B, hkv, sk, dv))
        if mx:
            (q8, k8, v8, qa, ka, va), (Qd, Kd, Vd) = _quantise(w, Q, K, V)
            o, lse = binding.forward_mxfp8(handle, dev(q8), dev(k8), dev(v8), dev(qa), dev(ka), dev(va), causal=causal, scale=w.scale)
        else:
            q8, sqs, Qd = W.quantize_e4m3_blocks(Q, 128)
            k8, sks, Kd = W.quantize_e4m3_blocks(K, 128)
            v8, svs, Vd = W.quantize_e4m3_blocks(V, None)
            o, lse = binding.forward_fp8(handle, dev(q8), dev(k8), dev(v8), dev(sqs), dev(sks), dev(svs), causal=causal, scale=w.scale)
        torch.cuda.synchronize()
        st, detail = binding.fa_last_status(handle)
        assert st == binding.FA_OK, (name, st, hex(detail))
        assert binding.fa_last_kernel_name(handle) == ("fa_fwd_mxfp8_stream" if mx else "fa_fwd_fp8_stream"), name
        splits_seen.add((mx, binding.fa_last_kv_splits(handle) > 1))
        O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=causal, scale=w.scale)
        _check(w, bf16_tensor_to_f64(o), lse.double().cpu().numpy(), O_ref, lse_ref, Vd, mean_bound=1e-2)
    assert splits_seen == {(True, False), (True, True), (False, False), (False, True)}, splits_seen
