"""GPU parity: the CUDA path, called through the C ABI, against the fp64 oracle, element by element."""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, run_gpu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def handles():
    from paper_2609_21264_b200 import binding
    hs = {"pipelined": binding.fa_create(), "serial": binding.fa_create(flags=binding.FA_FLAG_SERIAL_KERNEL),
          "persistent": binding.fa_create(flags=binding.FA_FLAG_FORCE_PERSISTENT | binding.FA_FLAG_NO_STREAM_KERNEL)}
    yield hs
    for h in hs.values():
        assert binding.fa_destroy(h) == binding.FA_OK


def _wl(name, B, Hq, Hkv, Sq, Sk, dqk, dv, causal, seed=1, sigma=1.0, k_mult=1.0, scale=None):
    return W.Workload(name, B, Hq, Hkv, Sq, Sk, dqk, dv, causal,
                      scale if scale is not None else dqk ** -0.5, sigma, k_mult, seed)


# Shapes the oracle finishes in a moment; they span several tiles, ragged tails, Sq != Sk,
# single rows/keys, GQA groups, all three head-size pairs, both mask modes.
SMALL = [
    _wl("one_tile_d64", 1, 1, 1, 128, 128, 64, 64, False),
    _wl("one_tile_d128", 1, 1, 1, 128, 128, 128, 128, False),
    _wl("one_tile_d192", 1, 1, 1, 128, 128, 192, 128, True),
    _wl("single_row_single_key", 1, 1, 1, 1, 1, 64, 64, False),
    _wl("single_row_many_keys", 2, 4, 2, 1, 300, 128, 128, True),
    _wl("many_rows_single_key", 1, 2, 1, 300, 1, 128, 128, False),
    _wl("ragged_d64", 2, 4, 2, 200, 333, 64, 64, True),
    _wl("ragged_d64_noncausal", 1, 3, 3, 257, 129, 64, 64, False),
    _wl("ragged_d128_sq_gt_sk", 1, 2, 2, 333, 200, 128, 128, True),   # rows without any visible key
    _wl("ragged_d128_noncausal", 1, 2, 1, 383, 641, 128, 128, False),
    _wl("ragged_d192", 1, 2, 2, 300, 300, 192, 128, True),
    _wl("ragged_d192_noncausal", 2, 2, 1, 130, 515, 192, 128, False),
    _wl("multi_tile_causal_gqa", 1, 8, 2, 1024, 1024, 128, 128, True),
    _wl("multi_tile_odd_tiles", 1, 2, 2, 640, 640, 128, 128, True),
    _wl("multi_tile_d64_causal", 1, 4, 4, 1152, 1152, 64, 64, True),
    _wl("decode_like", 1, 8, 2, 3, 2000, 128, 128, True),
    _wl("sharp_rows", 1, 2, 2, 512, 512, 128, 128, True, k_mult=4.0),
    _wl("large_sigma", 1, 2, 2, 384, 384, 64, 64, True, sigma=2.0),
    _wl("custom_scale", 1, 2, 2, 256, 256, 128, 128, False, scale=0.3),
]


@pytest.mark.parametrize("kernel", ["pipelined", "serial"])
@pytest.mark.parametrize("w", SMALL, ids=[w.name for w in SMALL])
def test_small_shapes_match_oracle(handles, kernel, w):
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    O, lse = run_gpu(handles[kernel], w, Q, K, V)
    tol_scale = 1.0
    if w.sigma > 1.0:
        tol_scale = w.sigma        # |O| grows with sigma; the bar is stated for sigma = 1
    e = assert_parity(O / tol_scale, lse, O_ref / tol_scale, lse_ref, w.name)
    if w.name == "ragged_d128_sq_gt_sk":
        assert np.isneginf(lse_ref).any()          # the degenerate rows are really exercised
        assert (O[np.isneginf(lse_ref)] == 0).all()


@pytest.mark.parametrize("idx", [0, 1])
def test_full_configs_all_rows(handles, idx):
    w = W.config(idx)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale)
    O, lse = run_gpu(handles["pipelined"], w, Q, K, V)
    assert_parity(O, lse, O_ref, lse_ref, w.name)


def _sampled(handles, w, n_random, heads):
    Q, K, V = W.make_inputs(w)
    O, lse = run_gpu(handles["pipelined"], w, Q, K, V)
    rows = W.sample_rows(w, n_random, seed=w.seed, heads=heads)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=w.causal, scale=w.scale, rows=rows)
    Og = O[rows[:, 0], rows[:, 1], rows[:, 2]]
    lg = lse[rows[:, 0], rows[:, 1], rows[:, 2]]
    assert_parity(Og, lg, O_ref, lse_ref, w.name)
    # properties that hold at any size: finite everywhere, row 0 of a causal problem is V[0]
    assert np.isfinite(O).all() and np.isfinite(lse).all()
    if w.causal and w.Sq == w.Sk:
        G = w.Hq // w.Hkv
        v0 = W.bf16_bits_to_f64(V[:, :, 0, :])
        np.testing.assert_array_equal(O[:, :, 0, :], np.repeat(v0, G, axis=1))


def _all_rows(handles, w, kernels=("pipelined",)):
    """Every row of every head of a full-size configuration against the oracle (head by head, to bound the memory),
    for the library's own choice of kernel and for any other handle named in `kernels`."""
    Q, K, V = W.make_inputs(w)
    outs = {name: run_gpu(handles[name], w, Q, K, V) for name in kernels}
    for O, lse in outs.values():
        assert np.isfinite(O).all() and np.isfinite(lse).all()
    G = w.Hq // w.Hkv
    worst = {"o_max": 0.0, "o_mean": 0.0, "lse_max": 0.0}
    for b in range(w.B):
        for h0 in range(0, w.Hq, 8):
            hs = slice(h0, min(h0 + 8, w.Hq))
            ks = slice(hs.start // G, (hs.stop - 1) // G + 1)
            Qs = np.ascontiguousarray(Q[b:b + 1, hs])
            # the K/V heads these query heads read; the head map is preserved when 8 is a multiple of the group size
            assert 8 % G == 0, "the slices of 8 query heads must hold whole groups"
            O_ref, lse_ref = oracle.attention(Qs, np.ascontiguousarray(K[b:b + 1, ks]), np.ascontiguousarray(V[b:b + 1, ks]),
                                              causal=w.causal, scale=w.scale)
            for name, (O, lse) in outs.items():
                e = assert_parity(O[b:b + 1, hs], lse[b:b + 1, hs], O_ref, lse_ref,
                                  "%s (%s) batch %d heads %d..%d" % (w.name, name, b, hs.start, hs.stop - 1))
                for k_ in worst:
                    worst[k_] = max(worst[k_], e[k_])
    return worst


def test_config3_llama2_7b_all_rows(handles):
    # 4 x 32 heads x 8192 rows: 4096 work items; every row of every item against the oracle, on the one-item-per-CTA
    # kernel the library picks and on the persistent kernel, whose ticket ring then hands out all 4096 items
    _all_rows(handles, W.config(2), kernels=("pipelined", "persistent"))


def test_config4_deepseek_v2_all_rows(handles):
    _all_rows(handles, W.config(3))


def test_config5_long_context_fixed_rows_of_every_head(handles):
    # 128K tokens: the oracle takes the fixed row set (tile-boundary rows, first, middle, last) of EVERY one of the 32
    # heads plus random rows; the properties that hold at any size are checked on the whole output
    _sampled(handles, W.config(4), 64, heads=None)


def test_serial_and_pipelined_kernels_agree(handles):
    w = _wl("agree", 1, 4, 2, 700, 900, 128, 128, True, seed=9)
    Q, K, V = W.make_inputs(w)
    O1, l1 = run_gpu(handles["pipelined"], w, Q, K, V)
    O2, l2 = run_gpu(handles["serial"], w, Q, K, V)
    assert np.abs(O1 - O2).max() <= 2e-2 and np.abs(l1 - l2).max() <= 1e-4


def test_repeated_launches_are_deterministic(handles):
    w = _wl("det", 1, 8, 2, 1024, 1024, 128, 128, True, seed=11)
    Q, K, V = W.make_inputs(w)
    O1, l1 = run_gpu(handles["pipelined"], w, Q, K, V)
    for _ in range(5):
        O2, l2 = run_gpu(handles["pipelined"], w, Q, K, V)
        np.testing.assert_array_equal(O1, O2)
        np.testing.assert_array_equal(l1, l2)


def test_host_buffer_entry_point(handles):
    import torch
    from paper_2609_21264_b200 import binding
    w = _wl("host", 1, 4, 2, 300, 300, 128, 128, True, seed=3)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=True, scale=w.scale)
    O = np.empty((1, 4, 300, 128), dtype=np.uint16)
    lse = np.empty((1, 4, 300), dtype=np.float32)
    st = binding.fa_forward_host(handles["pipelined"], Q.ctypes.data, K.ctypes.data, V.ctypes.data,
                                 O.ctypes.data, lse.ctypes.data, 1, 4, 2, 300, 300, 128, 128, True, w.scale,
                                 torch.cuda.current_stream().cuda_stream)
    assert st == binding.FA_OK
    assert_parity(W.bf16_bits_to_f64(O), lse.astype(np.float64), O_ref, lse_ref, "host")


def test_lse_may_be_null_and_scale_zero_means_default(handles):
    import torch
    from paper_2609_21264_b200 import binding
    w = _wl("nolse", 1, 2, 2, 256, 256, 64, 64, False, seed=4)
    Q, K, V = W.make_inputs(w)
    O_ref, lse_ref = oracle.attention(Q, K, V, causal=False, scale=64 ** -0.5)
    O, _ = run_gpu(handles["pipelined"], w.with_(scale=0.0), Q, K, V, want_lse=False)
    assert np.abs(O - O_ref).max() <= 2e-2


def test_argument_errors(handles):
    import torch
    from paper_2609_21264_b200 import binding as b
    h = handles["pipelined"]
    t = torch.zeros(1 * 2 * 128 * 128 + 8, dtype=torch.bfloat16, device="cuda")
    lse = torch.zeros(2 * 128, dtype=torch.float32, device="cuda")
    p = t.data_ptr()
    ok = dict(B=1, Hq=2, Hkv=2, Sq=128, Sk=128, dqk=128, dv=128)

    def call(Q=p, K=p, V=p, O=p, L=lse.data_ptr(), scale=0.1, **kw):
        a = dict(ok); a.update(kw)
        return b.fa_forward(h, Q, K, V, O, L, a["B"], a["Hq"], a["Hkv"], a["Sq"], a["Sk"], a["dqk"], a["dv"],
                            False, scale, 0)
    assert call(Q=None) == b.FA_ERR_INVALID_ARG
    assert call(O=None) == b.FA_ERR_INVALID_ARG
    assert call(Q=p + 2) == b.FA_ERR_INVALID_ARG            # misaligned
    assert call(Hq=3, Hkv=2) == b.FA_ERR_INVALID_ARG
    assert call(Sq=0) == b.FA_ERR_INVALID_ARG
    assert call(scale=float("nan")) == b.FA_ERR_INVALID_ARG
    assert call(scale=-1.0) == b.FA_ERR_INVALID_ARG
    assert call(dqk=96, dv=96) == b.FA_ERR_UNSUPPORTED
    assert call(dqk=128, dv=64) == b.FA_ERR_UNSUPPORTED
    assert b.fa_forward(None, p, p, p, p, None, 1, 2, 2, 128, 128, 128, 128, False, 0.1, 0) == b.FA_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert b.fa_last_status(h)[0] == b.FA_OK
    assert b.fa_destroy(None) == b.FA_OK
