"""Pins for the oracle's value quantizer, dequantizer, packing, query subspace and the
memory formula.  CPU only.  Each check is against a library routine (numpy float32
arithmetic, numpy SVD / eigh), a hand-computed bit pattern, or a number the paper prints.
"""
import os

import numpy as np
import pytest

import oracle
import squat_inputs as si

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


# ------------------------------------------------------------------ values (Section 2, Appendix C)
@pytest.mark.parametrize("bits,G,d", [(2, 32, 128), (4, 32, 128), (2, 128, 128), (4, 64, 128), (2, 8, 16)])
def test_values_match_numpy_float32(bits, G, d):
    rng = np.random.default_rng(bits * 100 + G)
    V = rng.standard_normal((257, d)).astype(np.float32)
    V[3] = 0.5                       # constant token: scale 0
    out = oracle.quant_values_f32(V, G, bits)
    L = np.float32(2 ** bits - 1)
    X = V.reshape(257, d // G, G)
    m, Mx = X.min(axis=2), X.max(axis=2)
    delta = (Mx - m) / L
    assert delta.dtype == np.float32
    with np.errstate(divide="ignore", invalid="ignore"):
        t = (X - m[..., None]) / delta[..., None]
    c = np.where(delta[..., None] > 0, np.clip(np.rint(t), 0, L), 0).astype(np.uint8)
    assert np.array_equal(out["codes"], c.reshape(257, d))
    assert np.array_equal(out["scale"], delta) and np.array_equal(out["zero"], m)
    assert out["scale"][3, 0] == 0 and not out["codes"][3].any()


def test_values_f64_differs_from_f32_only_near_ties():
    cfg = si.get_config(1)
    V = si.to_f32(si.gen_values_unit(cfg, 0, 0, 512), cfg.dtype)
    a = oracle.quant_values_f32(V, 32, 2)
    b = oracle.quant_values_f64(V.astype(np.float64), 32, 2)
    assert np.array_equal(a["zero"], b["zero"])
    assert np.abs(a["scale"].astype(np.float64) - b["scale"]).max() <= 1.2e-7 * np.abs(b["scale"]).max()
    # bf16 data is coarse enough to produce exact rounding ties; the two precisions may break
    # them differently, and nowhere else
    bad = a["codes"] != b["codes"]
    assert bad.mean() < 1e-3
    t = (V.astype(np.float64).reshape(512, 4, 32) - b["zero"][..., None]) / b["scale"][..., None].astype(np.float64)
    frac = np.abs(t - np.floor(t) - 0.5).reshape(512, 128)
    assert np.all(frac[bad] < 1e-6)
    assert np.all(np.abs(a["codes"].astype(int) - b["codes"].astype(int))[bad] == 1)


def test_value_extremes_hit_both_ends_of_the_grid():
    rng = np.random.default_rng(7)
    V = rng.standard_normal((64, 128)).astype(np.float32)
    out = oracle.quant_values_f32(V, 32, 2)
    c = out["codes"].reshape(64, 4, 32)
    assert np.all(c.min(axis=2) == 0) and np.all(c.max(axis=2) == 3)
    deq = oracle.dequant_values(out["codes"], out["scale"], out["zero"], 32)
    assert np.abs(deq - V).max() <= 0.5 * out["scale"].max() * (1 + 1e-6)


# ------------------------------------------------------------------ dequantize (Section 2, deq)
def test_dequant_layouts():
    rng = np.random.default_rng(8)
    n, d, G = 64, 32, 16
    codes = rng.integers(0, 4, (n, d), dtype=np.uint8)
    sk = rng.random((n // G, d), dtype=np.float32)
    zk = rng.standard_normal((n // G, d)).astype(np.float32)
    dk = oracle.dequant_keys(codes, sk, zk, G)
    ref = codes.astype(np.float64) * np.repeat(sk, G, axis=0).astype(np.float64) + np.repeat(zk, G, axis=0)
    assert np.array_equal(dk, ref)
    sv = rng.random((n, d // G), dtype=np.float32)
    zv = rng.standard_normal((n, d // G)).astype(np.float32)
    dv = oracle.dequant_values(codes, sv, zv, G)
    ref = codes.astype(np.float64) * np.repeat(sv, G, axis=1).astype(np.float64) + np.repeat(zv, G, axis=1)
    assert np.array_equal(dv, ref)


# ------------------------------------------------------------------ packing (our cache layout)
def test_pack_bit_positions_by_hand():
    codes = np.array([[1, 2, 3, 0, 0, 0, 0, 3]], dtype=np.uint8)
    assert oracle.pack(codes, 2).tolist() == [[1 | (2 << 2) | (3 << 4), 3 << 6]]
    codes4 = np.array([[0xA, 0x3, 0xF, 0x1]], dtype=np.uint8)
    assert oracle.pack(codes4, 4).tolist() == [[0x3A, 0x1F]]


@pytest.mark.parametrize("bits", [1, 2, 4, 8])
def test_pack_unpack_roundtrip_every_code_every_position(bits):
    d = 16
    rows = []
    for code in range(2 ** bits):
        for pos in range(d):
            row = np.zeros(d, dtype=np.uint8)
            row[pos] = code
            rows.append(row)
    codes = np.array(rows, dtype=np.uint8)
    packed = oracle.pack(codes, bits)
    assert packed.shape == (len(rows), d * bits // 8)
    assert np.array_equal(oracle.unpack(packed, d, bits), codes)
    rng = np.random.default_rng(bits)
    rnd = rng.integers(0, 2 ** bits, (100, 128), dtype=np.uint8)
    assert np.array_equal(oracle.unpack(oracle.pack(rnd, bits), 128, bits), rnd)


# ------------------------------------------------------------------ subspace (Section 3.2, Alg. 1 l.5-6)
@pytest.mark.parametrize("N,d,r", [(50, 16, 5), (300, 64, 20), (512, 128, 32), (20, 32, 8)])
def test_subspace_matches_library_svd(N, d, r):
    rng = np.random.default_rng(N + d)
    Q = rng.standard_normal((N, 6)) @ rng.standard_normal((6, d)) + 0.3 * rng.standard_normal((N, d))
    Qhat, mu, V = oracle.query_subspace(Q, r)
    _, s, vt = np.linalg.svd(Q, full_matrices=False)
    ref = (vt[:r].T * s[:r] ** 2) @ vt[:r]              # Qhat^T Qhat = sum_{i<=r} sigma_i^2 v_i v_i^T
    assert np.abs(Qhat.T @ Qhat - ref).max() < 1e-9 * s[0] ** 2
    k = min(N, d)
    assert np.allclose(np.sqrt(np.maximum(mu[:k], 0)), s[:k], rtol=1e-9, atol=1e-9 * s[0])
    assert np.all(np.diff(mu) <= 1e-9 * mu[0])
    # rows of Qhat are sigma_i v_i: mutually orthogonal with norms sigma_i
    Gm = Qhat @ Qhat.T
    assert np.allclose(np.diag(Gm), s[:r] ** 2, rtol=1e-9)
    assert np.abs(Gm - np.diag(np.diag(Gm))).max() < 1e-9 * s[0] ** 2


def test_subspace_of_exactly_low_rank_queries_captures_them():
    rng = np.random.default_rng(3)
    Q = rng.standard_normal((200, 5)) @ rng.standard_normal((5, 32))
    Qhat, mu, V = oracle.query_subspace(Q, 5)
    Vr = V[:5]
    assert np.linalg.norm(Q - Q @ Vr.T @ Vr) < 1e-9 * np.linalg.norm(Q)
    assert np.abs(mu[5:]).max() < 1e-9 * mu[0]


def test_jacobi_residuals_and_orthogonality():
    rng = np.random.default_rng(4)
    A = rng.standard_normal((128, 128))
    A = A @ A.T
    mu, V = oracle.jacobi_eig(A)
    assert np.abs(A @ V.T - V.T * mu).max() < 1e-12 * np.abs(mu).max()
    assert np.abs(V @ V.T - np.eye(128)).max() < 1e-12
    assert np.allclose(mu, np.linalg.eigvalsh(A)[::-1], rtol=1e-11, atol=1e-11 * mu[0])


def test_gram_matches_library():
    rng = np.random.default_rng(5)
    Q = rng.standard_normal((333, 24))
    assert np.allclose(oracle.gram(Q), Q.T @ Q, rtol=1e-13, atol=1e-12)


# ------------------------------------------------------------------ Appendix B worked example
def test_kv_memory_worked_example():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "kv_memory_example.txt")) if l.strip() and not l.startswith("#")]
    assert rows
    for b, s, L, h, d, p, expected in rows:
        assert oracle.kv_cache_bytes(int(b), int(s), int(L), int(h), int(d), int(p)) == int(expected)


def test_exact_ties_round_half_to_even():
    # grid m = 0, Delta = 1 (b = 2): 0.5 -> 0, 1.5 -> 2, 2.5 -> 2  (nearest integer, ties to even)
    row = np.array([0.0, 3.0, 0.5, 1.5, 2.5, 1.0, 2.0, 0.25], dtype=np.float32)
    expect = [0, 3, 0, 2, 2, 1, 2, 0]
    assert oracle.quant_values_f32(row[None, :], 8, 2)["codes"][0].tolist() == expect
    assert oracle.quant_values_f64(row[None, :].astype(np.float64), 8, 2)["codes"][0].tolist() == expect
    assert oracle.quant_keys(row[:, None].astype(np.float64), 8, 2, None)["codes"][:, 0].tolist() == expect
