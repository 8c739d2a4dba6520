"""Pins of the fp64 oracle against what the definition (Eq. 1) and mathematics fix.

None of these tests re-types the oracle's formula: they use closed forms,
invariants, special cases, and a structurally different brute-force
implementation (full score and probability matrices with numpy long double).
"""
import itertools
import json
import math
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rnd(shape, seed, scale=1.0):
    return np.random.default_rng(seed).standard_normal(shape) * scale


def brute_force(Q, K, V, causal, scale):
    """Materialise S and P for every head with long double; einsum contraction."""
    Q = Q.astype(np.longdouble); K = K.astype(np.longdouble); V = V.astype(np.longdouble)
    B, Hq, Sq, _ = Q.shape
    _, Hkv, Sk, dv = V.shape
    G = Hq // Hkv
    Kx = np.repeat(K, G, axis=1)
    Vx = np.repeat(V, G, axis=1)
    S = np.einsum("bhid,bhjd->bhij", Q, Kx) * np.longdouble(scale)
    if causal:
        i = np.arange(Sq)[:, None]
        j = np.arange(Sk)[None, :]
        S = np.where(j <= i + (Sk - Sq), S, -np.inf)
    with np.errstate(invalid="ignore", divide="ignore"):
        m = S.max(axis=-1, keepdims=True)
        m_safe = np.where(np.isfinite(m), m, 0)
        E = np.exp(S - m_safe)
        l = E.sum(axis=-1, keepdims=True)
        P = np.where(l > 0, E / np.where(l > 0, l, 1), 0)
        O = np.einsum("bhij,bhjc->bhic", P, Vx)
        lse = np.where(l[..., 0] > 0, m_safe[..., 0] + np.log(np.where(l > 0, l, 1))[..., 0], -np.inf)
    return O.astype(np.float64), lse.astype(np.float64), P.astype(np.float64)


def test_hand_computed_2x2_golden():
    g = json.load(open(os.path.join(GOLDEN, "two_by_two.json")))
    Q = np.array(g["Q"], dtype=np.float64).reshape(1, 1, 2, 2)
    K = np.array(g["K"], dtype=np.float64).reshape(1, 1, 2, 2)
    V = np.array(g["V"], dtype=np.float64).reshape(1, 1, 2, 2)
    for case in g["cases"]:
        O, lse = oracle.attention(Q, K, V, causal=case["causal"], scale=case["scale"])
        np.testing.assert_allclose(O[0, 0], np.array(case["O"]), rtol=0, atol=2e-15 * 4)
        np.testing.assert_allclose(lse[0, 0], np.array(case["lse"]), rtol=0, atol=2e-15)


def test_golden_2x2_matches_closed_form():
    # the stored numbers themselves are checked against e^c/(1+e^c), independent of the oracle
    g = json.load(open(os.path.join(GOLDEN, "two_by_two.json")))
    for case in g["cases"]:
        c = case["scale"]
        s = math.exp(c) / (1.0 + math.exp(c))
        row1 = [1 + 2 * s, 2 + 2 * s]
        row0 = [1.0, 2.0] if case["causal"] else [3 - 2 * s, 4 - 2 * s]
        assert np.allclose(case["O"], [row0, row1], rtol=0, atol=1e-14)
        lse0 = c if case["causal"] else math.log1p(math.exp(c))
        assert np.allclose(case["lse"], [lse0, math.log1p(math.exp(c))], rtol=0, atol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_rows_of_P_sum_to_one(causal):
    Q, K, V = rnd((1, 2, 7, 8), 1), rnd((1, 2, 9, 8), 2), rnd((1, 2, 9, 4), 3)
    for hq, i in itertools.product(range(2), range(7)):
        P, O, lse = oracle.attention_prow(Q, K, V, causal=causal, scale=0.3, b=0, hq=hq, i=i)
        assert abs(P.sum() - 1.0) < 1e-14
        assert (P >= 0).all()
        nvis = 9 if not causal else i + 9 - 7 + 1
        assert (P[nvis:] == 0).all() and (P[:nvis] > 0).all()
        # the O row is P @ V
        np.testing.assert_allclose(O, P @ V[0, hq], rtol=0, atol=1e-14)


@pytest.mark.parametrize("causal", [False, True])
def test_constant_V_returns_the_constant(causal):
    Q, K = rnd((2, 4, 11, 16), 4, 2.0), rnd((2, 2, 11, 16), 5, 2.0)
    V = np.full((2, 2, 11, 6), 3.25)
    O, _ = oracle.attention(Q, K, V, causal=causal, scale=0.25)
    np.testing.assert_allclose(O, 3.25, rtol=0, atol=1e-14)


def test_single_key_returns_its_value_row():
    Q, K, V = rnd((1, 3, 5, 8), 6), rnd((1, 3, 1, 8), 7), rnd((1, 3, 1, 4), 8)
    O, lse = oracle.attention(Q, K, V, causal=False, scale=0.5)
    for h in range(3):
        for i in range(5):
            np.testing.assert_array_equal(O[0, h, i], V[0, h, 0])
            assert lse[0, h, i] == pytest.approx(0.5 * Q[0, h, i] @ K[0, h, 0], abs=1e-14)
    # causal, Sq == Sk: row 0 sees key 0 only
    K2, V2 = rnd((1, 3, 5, 8), 9), rnd((1, 3, 5, 4), 10)
    O2, lse2 = oracle.attention(Q, K2, V2, causal=True, scale=0.5)
    for h in range(3):
        np.testing.assert_array_equal(O2[0, h, 0], V2[0, h, 0])
        assert lse2[0, h, 0] == pytest.approx(0.5 * Q[0, h, 0] @ K2[0, h, 0], abs=1e-14)


@pytest.mark.parametrize("Sq,Sk", [(6, 6), (4, 9), (9, 4)])
def test_zero_Q_gives_uniform_average(Sq, Sk):
    K, V = rnd((1, 1, Sk, 4), 11), rnd((1, 1, Sk, 3), 12)
    Q = np.zeros((1, 1, Sq, 4))
    O, lse = oracle.attention(Q, K, V, causal=False, scale=1.0)
    np.testing.assert_allclose(O[0, 0], np.broadcast_to(V[0, 0].mean(axis=0), (Sq, 3)), atol=1e-14)
    np.testing.assert_allclose(lse[0, 0], math.log(Sk), atol=1e-14)
    O, lse = oracle.attention(Q, K, V, causal=True, scale=1.0)
    for i in range(Sq):
        n = min(Sk, max(0, i + Sk - Sq + 1))   # bottom-right aligned causal mask
        if n == 0:
            assert (O[0, 0, i] == 0).all() and lse[0, 0, i] == -np.inf
        else:
            np.testing.assert_allclose(O[0, 0, i], V[0, 0, :n].mean(axis=0), atol=1e-14)
            assert lse[0, 0, i] == pytest.approx(math.log(n), abs=1e-14)


def test_masked_entries_contribute_nothing():
    S = 8
    Q, K, V = rnd((1, 2, S, 4), 13), rnd((1, 2, S, 4), 14), rnd((1, 2, S, 4), 15)
    O, lse = oracle.attention(Q, K, V, causal=True, scale=0.5)
    for i in range(S - 1):
        K2, V2 = K.copy(), V.copy()
        K2[:, :, i + 1:, :] = 1e4      # would dominate every softmax if visible
        V2[:, :, i + 1:, :] = -7e6
        O2, lse2 = oracle.attention(Q, K2, V2, causal=True, scale=0.5)
        np.testing.assert_array_equal(O2[:, :, : i + 1], O[:, :, : i + 1])
        np.testing.assert_array_equal(lse2[:, :, : i + 1], lse[:, :, : i + 1])
        assert not np.array_equal(O2[:, :, i + 1:], O[:, :, i + 1:])


def test_shift_invariance():
    Q, K, V = rnd((1, 2, 5, 8), 16), rnd((1, 2, 7, 8), 17), rnd((1, 2, 7, 4), 18)
    c = rnd((8,), 19, 3.0)
    O, lse = oracle.attention(Q, K, V, causal=False, scale=0.4)
    O2, lse2 = oracle.attention(Q, K + c, V, causal=False, scale=0.4)
    np.testing.assert_allclose(O2, O, rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse2 - lse, 0.4 * (Q @ c), rtol=0, atol=1e-13)


def test_key_permutation_invariance():
    Q, K, V = rnd((1, 2, 5, 8), 20), rnd((1, 2, 13, 8), 21), rnd((1, 2, 13, 4), 22)
    perm = np.random.default_rng(23).permutation(13)
    O, lse = oracle.attention(Q, K, V, causal=False, scale=0.7)
    O2, lse2 = oracle.attention(Q, K[:, :, perm], V[:, :, perm], causal=False, scale=0.7)
    np.testing.assert_allclose(O2, O, rtol=0, atol=1e-13)
    np.testing.assert_allclose(lse2, lse, rtol=0, atol=1e-13)


def test_split_merge_identity():
    # attention over [K1; K2] equals the lse-weighted merge of the two halves
    # (the corrected form of the partial-result merge of Algorithm 2)
    Q, K, V = rnd((1, 2, 6, 8), 24), rnd((1, 2, 10, 8), 25, 2.0), rnd((1, 2, 10, 5), 26)
    O, lse = oracle.attention(Q, K, V, causal=False, scale=0.35)
    O1, l1 = oracle.attention(Q, K[:, :, :4], V[:, :, :4], causal=False, scale=0.35)
    O2, l2 = oracle.attention(Q, K[:, :, 4:], V[:, :, 4:], causal=False, scale=0.35)
    lm = np.logaddexp(l1, l2)
    Om = np.exp(l1 - lm)[..., None] * O1 + np.exp(l2 - lm)[..., None] * O2
    np.testing.assert_allclose(Om, O, rtol=0, atol=1e-13)
    np.testing.assert_allclose(lm, lse, rtol=0, atol=1e-13)


def test_gqa_equals_mha_with_repeated_kv_heads():
    Q, K, V = rnd((2, 6, 5, 8), 27), rnd((2, 2, 7, 8), 28), rnd((2, 2, 7, 4), 29)
    O, lse = oracle.attention(Q, K, V, causal=True, scale=0.3)
    O2, lse2 = oracle.attention(Q, np.repeat(K, 3, axis=1), np.repeat(V, 3, axis=1), causal=True, scale=0.3)
    np.testing.assert_array_equal(O, O2)
    np.testing.assert_array_equal(lse, lse2)
    # heads 0..2 read kv head 0, heads 3..5 read kv head 1 (contiguous groups)
    K3 = K.copy(); K3[:, 1] += 1.0
    O3, _ = oracle.attention(Q, K3, V, causal=True, scale=0.3)
    np.testing.assert_array_equal(O3[:, :3], O[:, :3])
    assert not np.array_equal(O3[:, 3:], O[:, 3:])


def test_sharp_limit_picks_argmax_without_overflow():
    Q, K, V = rnd((1, 1, 4, 8), 30), rnd((1, 1, 9, 8), 31), rnd((1, 1, 9, 3), 32)
    scale = 1e4
    O, lse = oracle.attention(Q, K, V, causal=False, scale=scale)
    s = scale * (Q[0, 0] @ K[0, 0].T)
    assert np.isfinite(O).all() and np.isfinite(lse).all()
    for i in range(4):
        j = int(np.argmax(s[i]))
        np.testing.assert_allclose(O[0, 0, i], V[0, 0, j], atol=1e-12)
        assert lse[0, 0, i] == pytest.approx(s[i, j], rel=1e-14)


def test_brute_force_tiny_shapes():
    n = 0
    for B, (Hq, Hkv), Sq, Sk, (dqk, dv), causal in itertools.product(
            [1, 2], [(1, 1), (2, 1), (2, 2), (4, 2)], [1, 2, 3, 5, 8], [1, 2, 3, 5, 8],
            [(1, 1), (2, 4), (4, 2)], [False, True]):
        seed = 1000 + n
        Q, K, V = rnd((B, Hq, Sq, dqk), seed), rnd((B, Hkv, Sk, dqk), seed + 1), rnd((B, Hkv, Sk, dv), seed + 2)
        O, lse = oracle.attention(Q, K, V, causal=causal, scale=0.6)
        Ob, lb, _ = brute_force(Q, K, V, causal, 0.6)
        np.testing.assert_allclose(O, Ob, rtol=0, atol=1e-12)
        fin = np.isfinite(lb)
        np.testing.assert_array_equal(np.isfinite(lse), fin)
        np.testing.assert_allclose(lse[fin], lb[fin], rtol=0, atol=1e-12)
        n += 1
    assert n == 2 * 4 * 5 * 5 * 3 * 2


def test_bf16_inputs_are_widened_exactly_and_row_subsets_agree():
    from paper_2609_21264_b200 import workloads as W
    w = W.Workload("t", 2, 4, 2, 37, 53, 16, 8, True, 0.25, seed=5)
    Q, K, V = W.make_inputs(w)
    O, lse = oracle.attention(Q, K, V, causal=True, scale=w.scale)
    Of, lsef = oracle.attention(W.bf16_bits_to_f64(Q), W.bf16_bits_to_f64(K), W.bf16_bits_to_f64(V),
                                causal=True, scale=w.scale)
    np.testing.assert_array_equal(O, Of)
    np.testing.assert_array_equal(lse, lsef)
    rows = np.array([[0, 0, 0], [1, 3, 36], [1, 2, 17], [0, 1, 5]])
    Or, lr = oracle.attention(Q, K, V, causal=True, scale=w.scale, rows=rows)
    for r, (b, h, i) in enumerate(rows):
        np.testing.assert_array_equal(Or[r], O[b, h, i])
        assert lr[r] == lse[b, h, i]
    # and against brute force on a bigger, ragged shape
    Ob, lb, _ = brute_force(W.bf16_bits_to_f64(Q), W.bf16_bits_to_f64(K), W.bf16_bits_to_f64(V), True, w.scale)
    np.testing.assert_allclose(O, Ob, rtol=0, atol=1e-12)
    np.testing.assert_allclose(lse, lb, rtol=0, atol=1e-12)


def test_invalid_arguments_are_rejected():
    Q, K, V = rnd((1, 3, 2, 4), 1), rnd((1, 2, 2, 4), 2), rnd((1, 2, 2, 4), 3)
    with pytest.raises(ValueError):
        oracle.attention(Q, K, V, causal=False, scale=1.0)          # Hq % Hkv != 0
    with pytest.raises(TypeError):
        oracle.attention(Q.astype(np.float32), K, V, causal=False, scale=1.0)
    with pytest.raises(ValueError):
        oracle.attention(rnd((1, 2, 2, 4), 1), K, V, causal=False, scale=1.0, rows=[[0, 0, 2]])
