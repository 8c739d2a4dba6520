"""Seeded fuzz over the entry points (contiguous, strided, block-scaled 8-bit, packed batches): small
random problems of every kind through one default handle, each checked against the oracle, so that
whatever kernel, tiling, split count and head sharing the library plans for a shape is exercised;
and once more through a handle that takes the persistent kernel wherever it applies (small
problems would never reach it by themselves)."""
import numpy as np
import pytest

import oracle
from paper_2609_21264_b200 import workloads as W
from parity_util import to_torch_bf16, bf16_tensor_to_f64, errors, O_MAX_ABS, O_MEAN_ABS, LSE_MAX_ABS

pytestmark = pytest.mark.gpu
N_CASES = 160


@pytest.fixture(scope="module", params=["planned", "persistent_where_possible"])
def handle(request):
    from paper_2609_21264_b200 import binding
    h = binding.fa_create(flags=0 if request.param == "planned" else binding.FA_FLAG_FORCE_PERSISTENT)
    h_kind = request.param
    yield h, h_kind
    binding.fa_destroy(h)


def _check(handle, name, O, lse, O_ref, lse_ref, Vd=None, G=1):
    from paper_2609_21264_b200 import binding
    st, detail = binding.fa_last_status(handle)
    assert st == binding.FA_OK, (name, st, hex(detail))
    e = errors(O, lse, O_ref, lse_ref)
    assert np.isfinite(O).all(), name
    assert e["lse_max"] <= LSE_MAX_ABS and e["lse_inf_match"], (name, e)
    if Vd is not None:      # 8-bit path: bound of test_gpu_fp8.py
        vmax = np.abs(Vd).max(axis=(2, 3))
        bound = 2.0 ** -4 * np.repeat(vmax, G, axis=1)[:, :, None, None] + 2.0 ** -8 * np.abs(O_ref) + 1e-3
        assert (np.abs(O - O_ref) <= bound).all(), (name, e)
    else:
        assert e["o_max"] <= O_MAX_ABS and e["o_mean"] <= O_MEAN_ABS, (name, e)


def test_fuzz_all_entry_points(handle):
    import torch
    from paper_2609_21264_b200 import binding
    handle, handle_kind = handle
    rng = np.random.default_rng(20261127 if handle_kind == "planned" else 20261128)
    seen = set()
    for it in range(N_CASES):
        kind = int(rng.integers(0, 4))           # 0 contiguous, 1 [B,S,H,d] strides, 2 e4m3, 3 packed batch
        d = int(rng.choice([64, 128, 192])) if kind != 2 else int(rng.choice([64, 128]))
        dv = 128 if d == 192 else d
        hkv, gqa, B = int(rng.integers(1, 4)), int(rng.choice([1, 2, 3, 4, 6, 8])), int(rng.integers(1, 4))
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
        name = "case%d kind%d b%d h%dx%d %dx%d d%d %s" % (it, kind, B, hkv, gqa, sq, sk, d, "causal" if causal else "full")
        w = W.Workload(name, B=B, Hq=hkv * gqa, Hkv=hkv, Sq=sq, Sk=sk, dqk=d, dv=dv, causal=causal, scale=d ** -0.5, seed=30000 + it)
        Q, K, V = W.make_inputs(w)
        if kind in (0, 1):
            O_ref, lse_ref = oracle.attention(Q, K, V, causal=causal, scale=w.scale)
            q, k, v = to_torch_bf16(Q), to_torch_bf16(K), to_torch_bf16(V)
            if kind == 1:
                q, k, v = (x.transpose(1, 2).contiguous().transpose(1, 2) for x in (q, k, v))
            o, lse = binding.forward(handle, q, k, v, causal=causal, scale=w.scale)
            torch.cuda.synchronize()
            _check(handle, name, bf16_tensor_to_f64(o), lse.double().cpu().numpy(), O_ref, lse_ref)
        elif kind == 2:
            Qf, Kf, Vf = (W.bf16_bits_to_f64(x) for x in (Q, K, V))
            q8, sqs, Qd = W.quantize_e4m3_blocks(Qf, 128)
            k8, sks, Kd = W.quantize_e4m3_blocks(Kf, 128)
            v8, svs, Vd = W.quantize_e4m3_blocks(Vf, None)
            O_ref, lse_ref = oracle.attention(Qd, Kd, Vd, causal=causal, scale=w.scale)
            dev = lambda a: torch.from_numpy(a).cuda()
            o, lse = binding.forward_fp8(handle, dev(q8), dev(k8), dev(v8), dev(sqs), dev(sks), dev(svs), causal=causal, scale=w.scale)
            torch.cuda.synchronize()
            _check(handle, name, bf16_tensor_to_f64(o), lse.double().cpu().numpy(), O_ref, lse_ref, Vd=Vd, G=gqa)
        else:
            nb = int(rng.integers(1, 6))
            lq = [int(rng.integers(0, sq + 1)) for _ in range(nb)]
            lk = [int(rng.integers(0, sk + 1)) for _ in range(nb)]
            if max(lq) == 0:
                lq[0] = sq
            tq, tk = sum(lq), sum(lk)
            if tk == 0:
                continue
            ww = W.Workload("packed", B=1, Hq=hkv * gqa, Hkv=hkv, Sq=tq, Sk=tk, dqk=d, dv=dv, causal=False, scale=d ** -0.5, seed=40000 + it)
            Qp, Kp, Vp = W.make_inputs(ww)
            q = np.ascontiguousarray(Qp[0].transpose(1, 0, 2))
            k = np.ascontiguousarray(Kp[0].transpose(1, 0, 2))
            v = np.ascontiguousarray(Vp[0].transpose(1, 0, 2))
            cu_q = np.concatenate([[0], np.cumsum(lq)]).astype(np.int32)
            cu_k = np.concatenate([[0], np.cumsum(lk)]).astype(np.int32)
            o, lse = binding.forward_varlen(handle, to_torch_bf16(q), to_torch_bf16(k), to_torch_bf16(v), torch.from_numpy(cu_q).cuda(),
                                            torch.from_numpy(cu_k).cuda(), max(lq), causal=causal, scale=d ** -0.5)
            torch.cuda.synchronize()
            O, L = bf16_tensor_to_f64(o), lse.double().cpu().numpy()
            for b in range(nb):
                if lq[b] == 0:
                    continue
                qs, ks = slice(cu_q[b], cu_q[b + 1]), slice(cu_k[b], cu_k[b + 1])
                O_b, L_b = O[qs].transpose(1, 0, 2)[None], L[:, qs][None]
                if lk[b] == 0:
                    assert (O_b == 0).all() and np.isneginf(L_b).all(), name
                    continue
                O_ref, lse_ref = oracle.attention(np.ascontiguousarray(q[qs].transpose(1, 0, 2))[None],
                                                  np.ascontiguousarray(k[ks].transpose(1, 0, 2))[None],
                                                  np.ascontiguousarray(v[ks].transpose(1, 0, 2))[None], causal=causal, scale=d ** -0.5)
                _check(handle, name + " sequence %d (%d x %d)" % (b, lq[b], lk[b]), O_b, L_b, O_ref, lse_ref)
        seen.add((kind, binding.fa_last_kernel_name(handle), binding.fa_last_kv_splits(handle) > 1))
    # the fuzz is only worth its time if it reaches the tilings: both kernels of the 16-bit path, with and without
    # split-KV, the 8-bit stream kernel and packed batches on the stream kernel
    kernels = {(k, n) for k, n, _ in seen}
    if handle_kind == "planned":
        # (two query tiles per CTA: fa_fwd_pair at head size 128, fa_fwd_pipelined at the other head sizes)
        assert {(0, "fa_fwd_stream"), (0, "fa_fwd_pipelined"), (2, "fa_fwd_fp8_stream"), (3, "fa_fwd_stream")} <= kernels, seen
        assert "fa_fwd_pair" in {n for _, n in kernels}, seen
    else:
        # (fixed-length problems at 192/128, where the stream tiling is planned, run its persistent form under this handle,
        #  with fewer items than SMs as well as with several per SM)
        assert {(0, "fa_fwd_persistent"), (1, "fa_fwd_persistent"), (3, "fa_fwd_persistent"), (3, "fa_fwd_stream"),
                (0, "fa_fwd_stream_persistent"), (1, "fa_fwd_stream_persistent")} <= kernels, seen
    assert any(s for _, _, s in seen)
