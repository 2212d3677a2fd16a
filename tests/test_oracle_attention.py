"""CPU pins of the oracle's decode-step attention (Section 2, "(Masked) Attention mechanism"; the score
vector of the proof of Theorem 1) -- against things other than itself: a loop-by-loop restatement with
Python floats, closed forms, invariances of softmax, and the bound of Theorem 1."""
import math

import numpy as np
import pytest

import oracle

D = 128


def _quantized_unit(seed, n, bits=2, G=32, d=D):
    rng = np.random.default_rng(seed)
    K = rng.standard_normal((n, d))
    V = rng.standard_normal((n, d))
    kq = oracle.quant_keys(K, G, bits)                       # W = None: plain per-channel rounding
    vq = oracle.quant_values_f64(V, G, bits)
    return K, V, kq, vq


def test_attention_matches_a_loop_by_loop_restatement():
    rng = np.random.default_rng(0)
    n, d, nq = 7, 5, 2
    q, K, V = rng.standard_normal((nq, d)), rng.standard_normal((n, d)), rng.standard_normal((n, d))
    out = oracle.attention_decode(q, K, V)
    for h in range(nq):
        w = [sum(q[h][j] * K[i][j] for j in range(d)) / math.sqrt(d) for i in range(n)]
        e = [math.exp(x) for x in w]                         # no max subtraction here: same value by algebra
        z = sum(e)
        for j in range(d):
            ref = sum(e[i] / z * V[i][j] for i in range(n))
            assert abs(out[h][j] - ref) <= 1e-13 * max(1.0, abs(ref))


def test_zero_query_gives_the_mean_of_the_values():
    rng = np.random.default_rng(1)
    K, V = rng.standard_normal((40, D)), rng.standard_normal((40, D))
    out = oracle.attention_decode(np.zeros((1, D)), K, V)
    assert np.abs(out[0] - V.mean(axis=0)).max() <= 1e-14


def test_one_dominant_score_selects_that_value_row():
    rng = np.random.default_rng(2)
    K, V = rng.standard_normal((16, D)), rng.standard_normal((16, D))
    K[5] = 0.0
    K[5, 3] = 1.0
    q = np.zeros((1, D))
    q[0, 3] = 1e4                                            # w_5 = 1e4 / sqrt(d): every other weight underflows
    K[:, 3] = np.where(np.arange(16) == 5, 1.0, 0.0)
    out = oracle.attention_decode(q, K, V)
    assert np.array_equal(out[0], V[5])


def test_softmax_invariances():
    rng = np.random.default_rng(3)
    n = 33
    q, K, V = rng.standard_normal((3, D)), rng.standard_normal((n, D)), rng.standard_normal((n, D))
    out = oracle.attention_decode(q, K, V)
    # the same shift of every score leaves the weights unchanged: add a vector u to every key
    u = rng.standard_normal(D)
    out_shift = oracle.attention_decode(q, K + u, V)
    assert np.abs(out - out_shift).max() <= 1e-12
    # the order of the cached tokens does not matter
    perm = rng.permutation(n)
    assert np.abs(out - oracle.attention_decode(q, K[perm], V[perm])).max() <= 1e-13
    # query heads are independent
    for h in range(3):
        assert np.array_equal(out[h], oracle.attention_decode(q[h:h + 1], K, V)[0])
    # a convex combination of value rows: inside their per-channel range
    assert np.all(out <= V.max(axis=0) + 1e-12) and np.all(out >= V.min(axis=0) - 1e-12)


def test_scores_scale_with_one_over_sqrt_d():
    # d = 4, two tokens, scores 2/sqrt(4) = 1 and 0: weights e/(1+e), 1/(1+e)
    q = np.array([[2.0, 0, 0, 0]])
    K = np.array([[1.0, 0, 0, 0], [0, 0, 0, 0]])
    V = np.array([[1.0, 0, 0, 0], [0, 1.0, 0, 0]])
    out = oracle.attention_decode(q, K, V)
    p = math.e / (1 + math.e)
    assert abs(out[0, 0] - p) <= 1e-15 and abs(out[0, 1] - (1 - p)) <= 1e-15


@pytest.mark.parametrize("bits,G", [(2, 32), (4, 64)])
def test_attention_over_cache_composes_dequantization_and_residual(bits, G):
    n, R = 2 * G, 8
    K, V, kq, vq = _quantized_unit(4, n, bits, G)
    rng = np.random.default_rng(5)
    k_res, v_res = rng.standard_normal((R, D)), rng.standard_normal((R, D))
    q = rng.standard_normal((2, D))
    out = oracle.decode_attention_over_cache(q, kq["codes"], kq["scale"], kq["zero"], vq["codes"], vq["scale"],
                                             vq["zero"], G, k_res, v_res)
    # restated with numpy on arrays rebuilt from the codes by hand
    Kd = kq["codes"].astype(np.float64) * np.repeat(kq["scale"].astype(np.float64), G, axis=0) + \
        np.repeat(kq["zero"].astype(np.float64), G, axis=0)
    Vd = vq["codes"].astype(np.float64) * np.repeat(vq["scale"].astype(np.float64), G, axis=1) + \
        np.repeat(vq["zero"].astype(np.float64), G, axis=1)
    Kall, Vall = np.concatenate([Kd, k_res]), np.concatenate([Vd, v_res])
    w = q @ Kall.T / math.sqrt(D)
    p = np.exp(w - w.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    assert np.abs(out - p @ Vall).max() <= 1e-12
    # without a residual buffer the same call works on the quantized part alone
    out0 = oracle.decode_attention_over_cache(q, kq["codes"], kq["scale"], kq["zero"], vq["codes"], vq["scale"],
                                              vq["zero"], G)
    assert np.abs(out0 - oracle.attention_decode(q, Kd, Vd)).max() == 0.0


def test_theorem_1_bound_holds_for_the_quantized_cache():
    # Theorem 1: || Attn(q, K, V) - Attn(q, K^deq, V^deq) ||_2
    #   <= sum_i ||v_i - deq(v_i)|| / (2 sqrt(d)) * sum_i |q (k_i - deq(k_i))^T| + sum_i ||v_i - deq(v_i)||
    n, G, bits = 64, 32, 2
    K, V, kq, vq = _quantized_unit(6, n, bits, G)
    Kd = oracle.dequant_keys(kq["codes"], kq["scale"], kq["zero"], G)
    Vd = oracle.dequant_values(vq["codes"], vq["scale"], vq["zero"], G)
    rng = np.random.default_rng(7)
    for _ in range(5):
        q = rng.standard_normal((1, D))
        lhs = np.linalg.norm(oracle.attention_decode(q, K, V) - oracle.attention_decode(q, Kd, Vd))
        sv = np.linalg.norm(V - Vd, axis=1).sum()
        sk = np.abs((K - Kd) @ q[0]).sum()
        assert lhs <= sv / (2 * math.sqrt(D)) * sk + sv
        assert lhs > 0.0                                     # the bound is not vacuous: quantization does move the output
