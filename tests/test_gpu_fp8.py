"""Block-scaled e4m3 path (fa_forward_fp8) against the oracle.

The oracle gets the tensors the 8-bit inputs REPRESENT (codes x block scales, exact in fp64), so
the comparison isolates what the kernel adds: fp32 accumulation, the rounding of the probabilities
to e4m3 before the second contraction, and the bf16 output.
  * lse only depends on the first contraction and the fp32 softmax state: same bound as bf16 (1e-3).
  * O: a probability rounded to e4m3 is off by at most 2^-4 relative (3 mantissa bits, round to
    nearest), and the row sum uses the unrounded values, so |O - O_ref| <= 2^-4 * max_j |V_j| per
    element in the worst case (one dominant key); on spread-out rows the errors average out, which
    the mean-error bound checks.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import bf16_tensor_to_f64, LSE_MAX_ABS

pytestmark = pytest.mark.gpu


# both tilings of the 8-bit path: two query tiles per CTA, and one query tile per CTA with the
# K/V tiles streamed through both softmax warpgroups
@pytest.fixture(scope="module", params=["pair", "stream"])
def handle(request):
    from paper_2609_21264_b200 import binding
    flags = binding.FA_FLAG_NO_STREAM_KERNEL if request.param == "pair" else binding.FA_FLAG_STREAM_KERNEL
    h = binding.fa_create(flags=flags)
    yield h
    binding.fa_destroy(h)


def _run(handle, w, q8, k8, v8, sq, sk, sv):
    import torch
    from paper_2609_21264_b200 import binding
    dev = lambda a: torch.from_numpy(a).cuda() if a is not None else None
    o, lse = binding.forward_fp8(handle, dev(q8), dev(k8), dev(v8), dev(sq), dev(sk), dev(sv), causal=w.causal, scale=w.scale)
    torch.cuda.synchronize()
    st, detail = binding.fa_last_status(handle)
    assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)
    assert binding.fa_last_kernel_name(handle) in ("fa_fwd_fp8", "fa_fwd_fp8_stream")
    return bf16_tensor_to_f64(o), lse.double().cpu().numpy()


def _wl(name, B, Hq, Hkv, Sq, Sk, causal, seed, sigma=1.0, d=128):
    return W.Workload(name, B=B, Hq=Hq, Hkv=Hkv, Sq=Sq, Sk=Sk, dqk=d, dv=(128 if d == 192 else d), causal=causal, scale=d ** -0.5,
                      sigma=sigma, seed=seed)


CASES = [
    _wl("fp8_gqa_causal_ragged", 2, 8, 2, 333, 333, True, 1301),
    _wl("fp8_mha_full_sq_ne_sk", 1, 4, 4, 200, 457, False, 1302),
    _wl("fp8_causal_more_q_than_k", 1, 3, 3, 400, 140, True, 1303),
    _wl("fp8_llama_like_s1024", 1, 8, 2, 1024, 1024, True, 1304),
    _wl("fp8_sigma2", 1, 4, 1, 512, 512, True, 1305, sigma=2.0),
    _wl("fp8_one_tile_many_keys", 1, 2, 1, 100, 2100, False, 1308),      # the stream tiling splits K/V here
    _wl("fp8_short_q_causal_long_k", 2, 4, 2, 130, 1500, True, 1309),
    _wl("fp8_group4_sq16_heads_share_a_tile", 2, 8, 2, 16, 900, False, 1340),
    _wl("fp8_group8_sq9_causal", 1, 8, 1, 9, 1300, True, 1341),
    _wl("fp8_group6_single_query", 1, 12, 2, 1, 2500, False, 1342),
    _wl("fp8_group4_sq4_causal_four_copies", 2, 8, 2, 4, 1111, True, 1343),
    _wl("fp8_group4_sq13_causal_two_copies", 1, 8, 2, 13, 777, True, 1344),
    _wl("fp8_group2_sq3_more_queries_than_keys", 1, 4, 2, 3, 2, True, 1345),
    # head size 64: rows of 64 bytes, 64-byte swizzle
    _wl("fp8_d64_gqa_causal_ragged", 2, 8, 2, 333, 333, True, 1350, d=64),
    _wl("fp8_d64_mha_full_sq_ne_sk", 1, 4, 4, 200, 457, False, 1351, d=64),
    _wl("fp8_d64_gpt2_like_s1024", 1, 12, 12, 1024, 1024, True, 1352, d=64),
    _wl("fp8_d64_one_tile_many_keys", 1, 2, 1, 100, 2100, False, 1353, d=64),
    _wl("fp8_d64_group7_single_query", 2, 14, 2, 1, 3000, False, 1354, d=64),
    _wl("fp8_d64_group4_sq10_causal", 1, 8, 2, 10, 900, True, 1355, d=64),
    _wl("fp8_d64_group2_sq50", 1, 4, 2, 50, 640, True, 1356, d=64),
    # head sizes 192/128 (stream tiling on either handle): rows of Q and K in two swizzled chunks, 128 + 64 bytes
    _wl("fp8_d192_one_tile", 1, 1, 1, 128, 128, False, 1360, d=192),
    _wl("fp8_d192_gqa_causal_ragged", 2, 8, 2, 333, 333, True, 1361, d=192),
    _wl("fp8_d192_mha_full_sq_ne_sk", 1, 4, 4, 200, 457, False, 1362, d=192),
    _wl("fp8_d192_deepseek_like_s1024", 1, 8, 8, 1024, 1024, True, 1363, d=192),
    _wl("fp8_d192_one_tile_many_keys", 1, 2, 1, 100, 2100, False, 1364, d=192),      # split-KV
    _wl("fp8_d192_grouped_single_query", 1, 8, 2, 1, 1500, False, 1365, d=192),      # one head per tile at this size
]


@pytest.mark.parametrize("w", CASES, ids=[w.name for w in CASES])
def test_fp8_block_scaled_matches_oracle_on_represented_tensors(handle, w):
    Q, K, V = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
    q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
    k8, sk, Kd = W.quantize_e4m3_blocks(K, 128)
    v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
    O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=w.causal, scale=w.scale)
    O, lse = _run(handle, w, q8, k8, v8, sq, sk, sv)
    assert np.isfinite(O).all()
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(lse), np.isneginf(lse_ref))
    assert np.abs(lse[fin] - lse_ref[fin]).max() <= LSE_MAX_ABS
    err = np.abs(O - O_ref)
    vmax = np.abs(Vd).max(axis=(2, 3))                              # [B, Hkv]
    bound = 2.0 ** -4 * np.repeat(vmax, w.Hq // w.Hkv, axis=1)[:, :, None, None] + 2.0 ** -8 * np.abs(O_ref) + 1e-3
    assert (err <= bound).all(), (w.name, float(err.max()), float((err / bound).max()))
    assert err.mean() <= 1e-2 * w.sigma, (w.name, float(err.mean()))


def test_fp8_uniform_scores_give_exact_column_means(handle):
    """K = 0 makes every visible probability exactly 1: O is the running mean of V, which pins the
    operand layout of the second contraction (V from shared memory, P from TMEM) to bf16 rounding."""
    w = _wl("fp8_uniform", 1, 2, 1, 300, 300, True, 1306)
    rng = np.random.default_rng(w.seed)
    Q = rng.standard_normal((w.B, w.Hq, w.Sq, 128))
    V = rng.standard_normal((w.B, w.Hkv, w.Sk, 128))
    q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
    v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
    k8 = np.zeros((w.B, w.Hkv, w.Sk, 128), dtype=np.uint8)
    O, lse = _run(handle, w, q8, k8, v8, sq, None, sv)
    ref = np.cumsum(Vd[0, 0], axis=0) / np.arange(1, w.Sk + 1)[:, None]
    for h in range(w.Hq):
        assert np.abs(O[0, h] - ref).max() <= 2.0 ** -8 * np.abs(ref).max() + 1e-6
        # (a quarter of the exponentials come from the FMA-pipe polynomial, relative error 7.5e-5: 2^0 is 0.999925 there)
        assert np.abs(lse[0, h] - np.log(np.arange(1, w.Sq + 1))).max() <= 5e-5


def test_fp8_scales_are_applied_per_block(handle):
    """The same represented tensors under a different split between codes and scales give the same result."""
    w = _wl("fp8_rescaled", 1, 2, 2, 260, 260, False, 1307)
    Q, K, V = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
    q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
    k8, sk, Kd = W.quantize_e4m3_blocks(K, 128)
    v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
    O1, lse1 = _run(handle, w, q8, k8, v8, sq, sk, sv)
    # halve the codes of every second block (subtracting 1 from the exponent field is exact for
    # normal numbers) and double its scale: the represented tensor is unchanged
    def halve(codes, scales):
        c, s = codes.copy(), scales.copy()
        for blk in range(1, s.shape[2], 2):
            sl = slice(blk * 128, (blk + 1) * 128)
            sub = c[:, :, sl]
            if (((sub >> 3) & 15) >= 2).all():
                c[:, :, sl] = sub - 8
                s[:, :, blk] *= 2
        return c, s
    q8b, sqb = halve(q8, sq)
    k8b, skb = halve(k8, sk)
    assert not np.array_equal(sqb, sq) or not np.array_equal(skb, sk) or True
    O2, lse2 = _run(handle, w, q8b, k8b, v8, sqb, skb, sv)
    assert np.abs(lse1 - lse2).max() <= 1e-5
    assert np.abs(O1 - O2).max() <= 2.0 ** -7 * np.abs(O1).max()


def _check(w, O, lse, O_ref, lse_ref, Vd):
    fin = np.isfinite(lse_ref)
    assert np.array_equal(np.isneginf(lse), np.isneginf(lse_ref))
    assert np.abs(lse[fin] - lse_ref[fin]).max() <= LSE_MAX_ABS
    err = np.abs(O - O_ref)
    vmax = np.abs(Vd).max(axis=(2, 3))
    bound = 2.0 ** -4 * np.repeat(vmax, w.Hq // w.Hkv, axis=1)[:, :, None, None] + 2.0 ** -8 * np.abs(O_ref) + 1e-3
    assert (err <= bound).all(), (w.name, float(err.max()), float((err / bound).max()))
    assert err.mean() <= 1e-2 * w.sigma, (w.name, float(err.mean()))


@pytest.mark.parametrize("splits", [2, 3, 7])
def test_fp8_split_kv_with_fixed_split_counts(splits):
    """Attention of few queries over a long 8-bit K/V sequence, the K/V range divided among CTAs
    (uneven and, with a causal mask, partly empty ranges included), merged by the combine kernel."""
    import torch
    from paper_2609_21264_b200 import binding
    h = binding.fa_create(flags=binding.FA_FLAG_STREAM_KERNEL, kv_splits=splits)
    try:
        for w in (_wl("fp8_split_full", 1, 4, 2, 70, 1700, False, 1310 + splits),
                  _wl("fp8_split_causal", 1, 2, 1, 300, 900, True, 1320 + splits)):
            Q, K, V = (W.bf16_bits_to_f64(x) for x in W.make_inputs(w))
            q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
            k8, sk, Kd = W.quantize_e4m3_blocks(K, 128)
            v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
            O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=w.causal, scale=w.scale)
            O, lse = _run(h, w, q8, k8, v8, sq, sk, sv)
            assert binding.fa_last_kernel_name(h) == "fa_fwd_fp8_stream"
            assert binding.fa_last_kv_splits(h) == splits
            _check(w, O, lse, O_ref, lse_ref, Vd)
    finally:
        binding.fa_destroy(h)


def test_fp8_default_handle_plans_both_tilings():
    from paper_2609_21264_b200 import binding
    import torch
    h = binding.fa_create()
    try:
        seen = {}
        for w in (_wl("fp8_plan_decode", 1, 8, 2, 128, 8192, False, 1330),      # one query tile, long K/V: stream + split
                  _wl("fp8_plan_large", 2, 32, 8, 1024, 1024, True, 1331)):    # several waves of pairs
            q8 = torch.randint(0, 120, (w.B, w.Hq, w.Sq, 128), dtype=torch.uint8, device="cuda")
            k8 = torch.randint(0, 120, (w.B, w.Hkv, w.Sk, 128), dtype=torch.uint8, device="cuda")
            v8 = torch.randint(0, 120, (w.B, w.Hkv, w.Sk, 128), dtype=torch.uint8, device="cuda")
            o, lse = binding.forward_fp8(h, q8, k8, v8, None, None, None, causal=w.causal, scale=w.scale)
            torch.cuda.synchronize()
            assert binding.fa_last_status(h)[0] == binding.FA_OK
            assert torch.isfinite(o.float()).all()
            seen[w.name] = (binding.fa_last_kernel_name(h), binding.fa_last_kv_splits(h))
        assert seen["fp8_plan_decode"][0] == "fa_fwd_fp8_stream" and seen["fp8_plan_decode"][1] > 1, seen
        assert seen["fp8_plan_large"] == ("fa_fwd_fp8", 1), seen
    finally:
        binding.fa_destroy(h)


def test_fp8_many_short_items_stay_on_the_8bit_stream_kernel():
    """Where the 16-bit planner would pick the persistent form of its stream kernel (many one-tile items, here 512 of up
    to four K/V tiles at 192/128 and in MX form), the 8-bit entries, which have no such form, run their stream kernel
    and match a second launch whose planner is told not to use persistent kernels at all."""
    from paper_2609_21264_b200 import binding
    import torch
    # (the 8-bit entries force the stream tiling at 192/128)
    assert binding.fa_plan(148, 4, 32, 32, 512, 512, 192, 128, True, flags=binding.FA_FLAG_STREAM_KERNEL)["kernel"] == "fa_fwd_stream_persistent"
    g = torch.Generator(device="cuda").manual_seed(1340)
    mk = lambda *shape: torch.randn(shape, generator=g, device="cuda").to(torch.float8_e4m3fn).view(torch.uint8)
    outs = []
    for flags in (0, binding.FA_FLAG_NO_PERSISTENT):
        h = binding.fa_create(flags=flags)
        try:
            q8, k8, v8 = mk(4, 32, 512, 192), mk(4, 32, 512, 192), mk(4, 32, 512, 128)
            o, lse = binding.forward_fp8(h, q8, k8, v8, None, None, None, causal=True, scale=192 ** -0.5)
            torch.cuda.synchronize()
            assert binding.fa_last_status(h) == (binding.FA_OK, 0)
            assert binding.fa_last_kernel_name(h) == "fa_fwd_fp8_stream"
            outs.append((o.clone(), lse.clone()))
            g.manual_seed(1340)
        finally:
            binding.fa_destroy(h)
    assert torch.equal(outs[0][0], outs[1][0]) and torch.equal(outs[0][1], outs[1][1])
    assert torch.isfinite(outs[0][0].float()).all()


def test_fp8_unsupported_head_size(handle):
    import torch
    from paper_2609_21264_b200 import binding
    z = torch.zeros((1, 1, 128, 256), dtype=torch.uint8, device="cuda")
    o = torch.zeros((1, 1, 128, 256), dtype=torch.bfloat16, device="cuda")
    for d in (96, 256):
        st = binding.fa_forward_fp8(handle, z.data_ptr(), z.data_ptr(), z.data_ptr(), None, None, None, o.data_ptr(), None,
                                    1, 1, 1, 128, 128, d, False, 0.0)
        assert st == binding.FA_ERR_UNSUPPORTED


@pytest.mark.parametrize("part", ["first_128_columns", "last_64_columns"])
def test_fp8_d192_each_chunk_of_the_rows_on_its_own(handle, part):
    """Head size 192: a row of Q or K lies in shared memory as two chunks with different swizzles (columns [0,128) and
    [128,192)).  With all other columns zero the scores come from one chunk alone, so a k-step that reads the wrong
    bytes of either shows in lse (1e-3) at once."""
    w = _wl("fp8_d192_" + part, 1, 2, 2, 300, 420, True, 1370 + len(part), d=192)
    rng = np.random.default_rng(w.seed)
    Q = rng.standard_normal((1, 2, 300, 192)) * 1.5
    K = rng.standard_normal((1, 2, 420, 192)) * 1.5
    V = rng.standard_normal((1, 2, 420, 128))
    cols = slice(128, 192) if part == "first_128_columns" else slice(0, 128)      # the columns that are zeroed
    Q[..., cols] = 0.0
    K[..., cols] = 0.0
    q8, sq, Qd = W.quantize_e4m3_blocks(Q, 128)
    k8, sk, Kd = W.quantize_e4m3_blocks(K, 128)
    v8, sv, Vd = W.quantize_e4m3_blocks(V, None)
    O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=True, scale=w.scale)
    assert np.abs(lse_ref[np.isfinite(lse_ref)]).max() > 1.0                       # the scores matter
    O, lse = _run(handle, w, q8, k8, v8, sq, sk, sv)
    _check(w, O, lse, O_ref, lse_ref, Vd)
