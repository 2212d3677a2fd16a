"""CPU pins of the oracle's rotary position embedding (the reader side of the variant of Section 4 that quantizes
keys before the embedding) -- against things other than itself: explicit 2 x 2 rotations written with math.cos /
math.sin, position 0, norm preservation, the composition law, and the relative-position property of the scores."""
import math

import numpy as np

import oracle

D = 128


def test_rope_matches_explicit_rotations_of_each_channel_pair():
    rng = np.random.default_rng(0)
    d, base = 8, 10000.0
    X = rng.standard_normal((3, d))
    pos = np.array([0, 5, 1234])
    out = oracle.rope_rows(X, pos, base)
    for t in range(3):
        for i in range(d // 2):
            a = pos[t] * base ** (-2.0 * i / d)                 # angle of pair (i, i + d/2)
            c, s = math.cos(a), math.sin(a)
            x0, x1 = X[t, i], X[t, i + d // 2]
            assert abs(out[t, i] - (x0 * c - x1 * s)) <= 1e-13
            assert abs(out[t, i + d // 2] - (x0 * s + x1 * c)) <= 1e-13
    # the first pair turns by exactly pos radians (base^0 = 1): a quarter turn maps (1, 0) to (0, 1) up to rounding
    e = np.zeros((1, d))
    e[0, 0] = 1.0
    q = oracle.rope_rows(e, np.array([1]), base)
    assert abs(q[0, 0] - math.cos(1.0)) <= 1e-15 and abs(q[0, d // 2] - math.sin(1.0)) <= 1e-15


def test_position_zero_is_the_identity_and_norms_are_kept():
    rng = np.random.default_rng(1)
    X = rng.standard_normal((5, D))
    assert np.array_equal(oracle.rope_rows(X, np.zeros(5, dtype=np.int64)), X)
    Y = oracle.rope_rows(X, np.array([1, 17, 300, 4095, 32767]))
    assert np.abs(np.linalg.norm(Y, axis=1) - np.linalg.norm(X, axis=1)).max() <= 1e-12
    # pairs do not mix: the squared length of every (i, i + d/2) pair is kept
    assert np.abs((Y[:, :64] ** 2 + Y[:, 64:] ** 2) - (X[:, :64] ** 2 + X[:, 64:] ** 2)).max() <= 1e-12
    assert not np.allclose(Y, X)


def test_rotations_compose_and_scores_depend_on_relative_position_only():
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal((1, D)), rng.standard_normal((1, D))
    # R(a) R(b) = R(a + b)
    twice = oracle.rope_rows(oracle.rope_rows(k, np.array([100])), np.array([23]))
    once = oracle.rope_rows(k, np.array([123]))
    assert np.abs(twice - once).max() <= 1e-12
    # <R(m) q, R(n) k> = <R(m - n) q, k>: shifting both positions by the same amount changes nothing
    s0 = float(oracle.rope_rows(q, np.array([900]))[0] @ oracle.rope_rows(k, np.array([400]))[0])
    s1 = float(oracle.rope_rows(q, np.array([900 + 77]))[0] @ oracle.rope_rows(k, np.array([400 + 77]))[0])
    s2 = float(oracle.rope_rows(q, np.array([500]))[0] @ k[0])
    assert abs(s0 - s1) <= 1e-10 and abs(s0 - s2) <= 1e-10


def test_attention_over_a_pre_rope_cache_composes_dequantization_rotation_and_attention():
    rng = np.random.default_rng(3)
    n, G, bits, R, first = 64, 32, 2, 5, 96
    K, V = rng.standard_normal((n, D)), rng.standard_normal((n, D))
    kq = oracle.quant_keys(K, G, bits)
    vq = oracle.quant_values_f64(V, G, bits)
    k_res, v_res = rng.standard_normal((R, D)), rng.standard_normal((R, D))
    q = rng.standard_normal((2, D))
    out = oracle.decode_attention_over_pre_rope_cache(q, kq["codes"], kq["scale"], kq["zero"], vq["codes"], vq["scale"],
                                                      vq["zero"], G, first, k_res, v_res)
    # restated with numpy: rotation written as a complex multiplication of the (i, i + 64) pairs
    Kd = np.concatenate([oracle.dequant_keys(kq["codes"], kq["scale"], kq["zero"], G), k_res])
    Vd = np.concatenate([oracle.dequant_values(vq["codes"], vq["scale"], vq["zero"], G), v_res])
    theta = 10000.0 ** (-2.0 * np.arange(64) / D)
    ang = (first + np.arange(n + R))[:, None] * theta[None, :]
    z = (Kd[:, :64] + 1j * Kd[:, 64:]) * np.exp(1j * ang)
    Kr = np.concatenate([z.real, z.imag], axis=1)
    w = q @ Kr.T / math.sqrt(D)
    p = np.exp(w - w.max(axis=1, keepdims=True))
    p /= p.sum(axis=1, keepdims=True)
    assert np.abs(out - p @ Vd).max() <= 1e-12
    # position matters: the same cache read as if it started at another position gives another result ...
    other = oracle.decode_attention_over_pre_rope_cache(q, kq["codes"], kq["scale"], kq["zero"], vq["codes"],
                                                        vq["scale"], vq["zero"], G, first + 32, k_res, v_res)
    assert np.abs(other - out).max() > 1e-3
    # ... and with every position 0 it is the plain reader
    plain = oracle.decode_attention_over_cache(q, kq["codes"], kq["scale"], kq["zero"], vq["codes"], vq["scale"],
                                               vq["zero"], G, k_res, v_res)
    Kall = np.concatenate([oracle.dequant_keys(kq["codes"], kq["scale"], kq["zero"], G), k_res])
    assert np.abs(oracle.attention_decode(q, oracle.rope_rows(Kall, np.zeros(n + R, dtype=np.int64)), Vd) - plain).max() == 0.0
