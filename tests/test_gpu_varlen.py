"""fa_forward_varlen: packed batches of sequences of different lengths against the oracle, sequence by sequence.

The oracle only knows one fixed-length problem, so every sequence of the batch is cut out of the
packed tensors and given to it on its own; the GPU sees the packed batch in one call.
"""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import assert_parity, bf16_tensor_to_f64, to_torch_bf16

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", params=["pipelined", "serial", "stream", "persistent"])
def handle(request):
    from paper_2609_21264_b200 import binding
    # the fixed-length comparison below wants the same tiling (hence rounding order) as the packed path
    flags = {"serial": binding.FA_FLAG_SERIAL_KERNEL, "pipelined": binding.FA_FLAG_NO_STREAM_KERNEL | binding.FA_FLAG_NO_PERSISTENT,
             "stream": binding.FA_FLAG_STREAM_KERNEL,
             "persistent": binding.FA_FLAG_NO_STREAM_KERNEL | binding.FA_FLAG_FORCE_PERSISTENT}[request.param]
    h = binding.fa_create(flags=flags)
    yield h
    binding.fa_destroy(h)


def _packed_inputs(lens_q, lens_k, Hq, Hkv, dqk, dv, seed):
    """Packed [total, H, d] bf16 bit tensors drawn with the recipe of the fixed-length workloads."""
    tq, tk = int(sum(lens_q)), int(sum(lens_k))
    w = W.Workload("packed", B=1, Hq=Hq, Hkv=Hkv, Sq=max(tq, 1), Sk=max(tk, 1), dqk=dqk, dv=dv,
                   causal=False, scale=dqk ** -0.5, seed=seed)
    Q, K, V = W.make_inputs(w)           # [1, H, S, d]
    q = np.ascontiguousarray(Q[0].transpose(1, 0, 2))[:tq]
    k = np.ascontiguousarray(K[0].transpose(1, 0, 2))[:tk]
    v = np.ascontiguousarray(V[0].transpose(1, 0, 2))[:tk]
    return q, k, v


def _run_and_check(handle, lens_q, lens_k, Hq, Hkv, dqk, dv, causal, seed, max_sq=None):
    import torch
    from paper_2609_21264_b200 import binding
    q, k, v = _packed_inputs(lens_q, lens_k, Hq, Hkv, dqk, dv, seed)
    cu_q = np.concatenate([[0], np.cumsum(lens_q)]).astype(np.int32)
    cu_k = np.concatenate([[0], np.cumsum(lens_k)]).astype(np.int32)
    tq, tk = q.shape[0], k.shape[0]
    dq = to_torch_bf16(q) if tq else torch.empty((0, Hq, dqk), dtype=torch.bfloat16, device="cuda")
    dk = to_torch_bf16(k) if tk else torch.empty((0, Hkv, dqk), dtype=torch.bfloat16, device="cuda")
    dv_ = to_torch_bf16(v) if tk else torch.empty((0, Hkv, dv), dtype=torch.bfloat16, device="cuda")
    if tk == 0:   # the call wants non-null pointers even for empty K/V
        dk = torch.zeros((1, Hkv, dqk), dtype=torch.bfloat16, device="cuda")[:0]
        dv_ = torch.zeros((1, Hkv, dv), dtype=torch.bfloat16, device="cuda")[:0]
    o, lse = binding.forward_varlen(handle, dq, dk, dv_, torch.from_numpy(cu_q).cuda(), torch.from_numpy(cu_k).cuda(),
                                    max(lens_q) if max_sq is None else max_sq, causal=causal, scale=dqk ** -0.5)
    torch.cuda.synchronize()
    st, detail = binding.fa_last_status(handle)
    assert st == binding.FA_OK, "device status %d (site 0x%x)" % (st, detail)
    O = bf16_tensor_to_f64(o) if tq else np.zeros((0, Hq, dv))
    L = lse.double().cpu().numpy()
    for b, (sq, sk) in enumerate(zip(lens_q, lens_k)):
        if sq == 0:
            continue
        qs, ks = slice(cu_q[b], cu_q[b + 1]), slice(cu_k[b], cu_k[b + 1])
        O_b = O[qs].transpose(1, 0, 2)[None]
        L_b = L[:, qs][None]
        if sk == 0:
            assert (O_b == 0).all() and np.isneginf(L_b).all()
            continue
        Qb = np.ascontiguousarray(q[qs].transpose(1, 0, 2))[None]
        Kb = np.ascontiguousarray(k[ks].transpose(1, 0, 2))[None]
        Vb = np.ascontiguousarray(v[ks].transpose(1, 0, 2))[None]
        O_ref, lse_ref = oracle.attention(Qb, Kb, Vb, causal=causal, scale=dqk ** -0.5)
        assert_parity(O_b, L_b, O_ref, lse_ref, "seq %d (%d x %d)" % (b, sq, sk))
    return O, L


@pytest.mark.parametrize("causal", [False, True], ids=["full", "causal"])
def test_self_attention_length_mix(handle, causal):
    lens = [1, 127, 128, 129, 300, 512, 57]
    _run_and_check(handle, lens, lens, Hq=4, Hkv=2, dqk=128, dv=128, causal=causal, seed=1101)


@pytest.mark.parametrize("dqk,dv", [(64, 64), (192, 128)], ids=["d64", "d192_128"])
def test_other_head_sizes(handle, dqk, dv):
    lens = [260, 31, 129]
    _run_and_check(handle, lens, lens, Hq=3, Hkv=3, dqk=dqk, dv=dv, causal=True, seed=1102)


def test_cross_lengths_and_empty_sequences(handle):
    """Sq_b != Sk_b (end-aligned causal mask), a sequence with no queries and one with no keys."""
    lens_q = [40, 0, 200, 130, 5]
    lens_k = [333, 50, 200, 0, 700]
    _run_and_check(handle, lens_q, lens_k, Hq=4, Hkv=1, dqk=128, dv=128, causal=True, seed=1103)
    _run_and_check(handle, lens_q, lens_k, Hq=4, Hkv=1, dqk=128, dv=128, causal=False, seed=1104)


def test_more_queries_than_keys_causal(handle):
    lens_q = [300, 64]
    lens_k = [100, 200]
    _run_and_check(handle, lens_q, lens_k, Hq=2, Hkv=2, dqk=64, dv=64, causal=True, seed=1105)


def test_one_sequence_equals_fixed_length_call(handle):
    """A batch of one sequence is the fixed-length problem in [S,H,d] layout: same bits as fa_forward."""
    import torch
    from paper_2609_21264_b200 import binding
    S, Hq, Hkv, d = 391, 4, 2, 128
    O, L = _run_and_check(handle, [S], [S], Hq=Hq, Hkv=Hkv, dqk=d, dv=d, causal=True, seed=1106)
    q, k, v = _packed_inputs([S], [S], Hq, Hkv, d, d, 1106)
    tq, tk, tv = (to_torch_bf16(np.ascontiguousarray(x.transpose(1, 0, 2))[None]) for x in (q, k, v))
    o, lse = binding.forward(handle, tq, tk, tv, causal=True, scale=d ** -0.5)
    torch.cuda.synchronize()
    assert np.array_equal(bf16_tensor_to_f64(o)[0].transpose(1, 0, 2), O)
    assert np.array_equal(lse.double().cpu().numpy()[0], L)


def test_rows_past_max_sq_are_left_alone_and_empty_batch(handle):
    import torch
    from paper_2609_21264_b200 import binding
    z = torch.zeros((8, 1, 64), dtype=torch.bfloat16, device="cuda")
    cu = torch.tensor([0, 8], dtype=torch.int32, device="cuda")
    args = (handle, z.data_ptr(), z.data_ptr(), z.data_ptr(), z.data_ptr(), None, cu.data_ptr(), cu.data_ptr())
    assert binding.fa_forward_varlen(*args, 0, 0, 0, 0, 1, 1, 64, 64, False, 0.0) == binding.FA_OK
    assert binding.fa_forward_varlen(*args, 1, 8, 8, 9, 1, 1, 64, 64, False, 0.0) == binding.FA_ERR_INVALID_ARG
    assert binding.fa_forward_varlen(*args[:6], None, cu.data_ptr(), 1, 8, 8, 8, 1, 1, 64, 64, False, 0.0) \
        == binding.FA_ERR_INVALID_ARG
    torch.cuda.synchronize()


@pytest.mark.parametrize("dqk,dv,Hq,Hkv", [(128, 128, 8, 2), (64, 64, 6, 2), (192, 128, 16, 1)], ids=["d128_g4", "d64_g3", "d192_g16"])
@pytest.mark.parametrize("causal", [False, True], ids=["full", "causal"])
def test_decode_batches_with_grouped_heads(handle, dqk, dv, Hq, Hkv, causal):
    """Few queries per sequence (here at most 40, lengths differing per sequence) against K/V of very
    different lengths, several query heads per K/V head: on the stream tiling the heads of a group
    share a query tile, each head's rows max_sq apart, and a sequence with fewer queries leaves
    the rest of its rows unused.  Includes a sequence without queries and one without keys."""
    from paper_2609_21264_b200 import binding
    lens_q = [1, 40, 7, 0, 16, 3, 1]
    lens_k = [900, 333, 1500, 64, 20, 0, 129]
    _run_and_check(handle, lens_q, lens_k, Hq=Hq, Hkv=Hkv, dqk=dqk, dv=dv, causal=causal, seed=1110 + dqk)
    # single-token decode for every sequence
    _run_and_check(handle, [1] * 9, [50, 700, 128, 129, 1, 2048, 300, 64, 1000], Hq=Hq, Hkv=Hkv, dqk=dqk, dv=dv,
                   causal=causal, seed=1120 + dqk)


def test_decode_batches_plan_shared_query_tiles():
    from paper_2609_21264_b200 import binding
    p = binding.fa_plan(148, 32, 32, 8, 1, 4096, 128, 128, True, varlen=True)
    assert p["kernel"] == "fa_fwd_stream" and p["heads_per_tile"] == 4 and p["kv_splits"] == 1 and p["ctas"] == 32 * 8
    assert binding.fa_plan(148, 32, 32, 8, 1, 4096, 128, 128, True, varlen=True,
                           flags=binding.FA_FLAG_NO_HEAD_PACKING)["heads_per_tile"] == 1


@pytest.mark.parametrize("splits", [0, 3, 5], ids=["auto", "3_splits", "5_splits"])
@pytest.mark.parametrize("grouped", [True, False], ids=["grouped_heads", "one_head_per_kv_head"])
def test_small_decode_batches_split_the_kv_range(splits, grouped):
    """A few sequences with one query tile each leave most SMs without work: the K/V range of every
    sequence is cut into C shares by its own CTAs (the lengths are only known on the device),
    the partials are merged by the combine kernel.  Includes an empty K/V sequence, a sequence
    with fewer tiles than shares, and a causal mask."""
    from paper_2609_21264_b200 import binding
    h = binding.fa_create(flags=binding.FA_FLAG_STREAM_KERNEL, kv_splits=splits)
    try:
        Hq, Hkv = (8, 2) if grouped else (4, 4)
        for causal in (False, True):
            _run_and_check(h, [1, 5, 1, 30], [4000, 130, 0, 2500], Hq=Hq, Hkv=Hkv, dqk=128, dv=128, causal=causal, seed=1130 + splits)
            assert binding.fa_last_kernel_name(h) == "fa_fwd_stream"
            if splits:
                assert binding.fa_last_kv_splits(h) == splits
            else:
                assert binding.fa_last_kv_splits(h) > 1
        _run_and_check(h, [100, 128, 7], [3000, 1500, 700], Hq=Hq, Hkv=Hkv, dqk=64, dv=64, causal=True, seed=1140 + splits)
    finally:
        binding.fa_destroy(h)
