"""Pins for the oracle's key quantizer (Algorithm 1, function Quant).

CPU only; the CUDA library is not involved.  The checks use what the mathematics fixes:
the lambda = 0 reduction to round-to-nearest, the closed form residual = (I + W) e with
every e a legal rounding error on the grid the algorithm must have chosen, a step-by-step
numerical solve of Eq. (2), exhaustive search on tiny problems, idempotence and chunking.
"""
import itertools

import numpy as np
import pytest

import oracle
import squat_inputs as si


def _case(seed, n, d, r, lam, g=1, n_q=200, outliers=True):
    rng = np.random.default_rng(seed)
    Qc = rng.standard_normal((n_q, max(r, 2))) @ rng.standard_normal((max(r, 2), d)) + 0.1 * rng.standard_normal((n_q, d))
    K = rng.standard_normal((n, d))
    if outliers and d >= 8:
        K[:, rng.choice(d, 2, replace=False)] *= 10
    mats = oracle.build_W(Qc, r, lam, g)
    return K, mats


def _rtn_per_channel(K, G, bits):
    """Textbook asymmetric round-to-nearest per channel over groups of G tokens."""
    n, d = K.shape
    L = 2 ** bits - 1
    X = K.reshape(n // G, G, d)
    m = X.min(axis=1)
    Mx = X.max(axis=1)
    zf = m.astype(np.float32)
    sf = ((Mx - m) / L).astype(np.float32)
    with np.errstate(divide="ignore", invalid="ignore"):
        t = (X - zf[:, None, :].astype(np.float64)) / sf[:, None, :].astype(np.float64)
    c = np.clip(np.rint(t), 0, L)
    c = np.where(sf[:, None, :] > 0, c, 0)
    return c.reshape(n, d).astype(np.uint8), sf, zf


@pytest.mark.parametrize("bits,G", [(2, 32), (4, 32), (2, 64), (3, 8)])
def test_lambda_zero_reduces_to_round_to_nearest(bits, G):
    K, mats = _case(1, 4 * G, 32, 4, 0.0)
    assert not mats["W"].any()
    out = oracle.quant_keys(K, G, bits, mats["W"])
    c, sf, zf = _rtn_per_channel(K, G, bits)
    assert np.array_equal(out["codes"], c)
    assert np.array_equal(out["scale"], sf) and np.array_equal(out["zero"], zf)
    out_none = oracle.quant_keys(K, G, bits, None)
    assert np.array_equal(out_none["codes"], c)


def test_rank_zero_reduces_to_round_to_nearest_with_exact_grid():
    # r = 0 and the plain definition with the grid in double: same codes (no element of this
    # seeded case sits within 1e-6 of a rounding midpoint, which is asserted).
    K, mats = _case(2, 64, 16, 0, 1e-3)
    out = oracle.quant_keys(K, 32, 2, mats["W"])
    X = K.reshape(2, 32, 16)
    m, Mx = X.min(axis=1, keepdims=True), X.max(axis=1, keepdims=True)
    t = (X - m) / ((Mx - m) / 3)
    assert np.abs(np.abs(t - np.floor(t)) - 0.5).min() > 1e-6
    assert np.array_equal(out["codes"], np.rint(t).reshape(64, 16).astype(np.uint8))


@pytest.mark.parametrize("d,r,g,bits,G", [(32, 4, 1, 2, 32), (32, 8, 8, 2, 16), (128, 32, 1, 2, 32), (128, 8, 32, 4, 32), (128, 16, 64, 2, 32)])
def test_residual_closed_form_and_grid(d, r, g, bits, G):
    # residual = (I + W) e, where e_j is the rounding error committed at channel j.  Recover e by a
    # triangular solve and check: (a) every |e| <= scale/2 (it IS a rounding error on that grid),
    # (b) the grid of channel j is min / (max-min)/L of the corrected values K + W e, (c) codes are
    # the rounding of those corrected values, (d) delta^T P delta = e^T D^-1 e with D from a library
    # Cholesky of P_inv.  A dropped term, wrong sign or transposed W breaks (a)-(c).
    lam = 1e-3 if d == 128 else 0.05
    K, mats = _case(3 + d + g, 2 * G, d, r, lam, g)
    W, P = mats["W"], mats["P"]
    out = oracle.quant_keys(K, G, bits, W)
    L = 2 ** bits - 1
    delta = out["Khat"] - K
    e = np.linalg.solve(np.eye(d) + W, delta.T).T
    X = K + e @ W.T                                  # value of channel j when it was quantized
    Xg = X.reshape(-1, G, d)
    sc = out["scale"].astype(np.float64)
    zr = out["zero"].astype(np.float64)
    assert np.all(np.abs(e.reshape(-1, G, d)) <= 0.5 * sc[:, None, :] * (1 + 1e-6) + 1e-12)
    assert np.allclose(Xg.min(axis=1), zr, rtol=1e-6, atol=1e-9)
    assert np.allclose((Xg.max(axis=1) - Xg.min(axis=1)) / L, sc, rtol=1e-6, atol=1e-9)
    t = (Xg - zr[:, None, :]) / sc[:, None, :]
    far = np.abs(np.abs(t - np.floor(t)) - 0.5) > 1e-6
    assert np.array_equal(np.clip(np.rint(t), 0, L)[far], out["codes"].reshape(-1, G, d)[far])
    assert np.allclose(out["Khat"].reshape(-1, G, d), zr[:, None, :] + sc[:, None, :] * out["codes"].reshape(-1, G, d))
    if g == 1:
        Dinv = 1.0 / np.diag(np.linalg.cholesky(np.linalg.inv(P))) ** 2
        lhs = np.einsum("ij,jk,ik->i", delta, P, delta)
        rhs = (e * e) @ Dinv
        assert np.allclose(lhs, rhs, rtol=1e-9)


@pytest.mark.parametrize("d,g,r,G,bits,lam", [(6, 1, 2, 3, 2, 0.5), (8, 2, 3, 4, 2, 0.1), (8, 1, 1, 2, 1, 2.0), (8, 4, 3, 4, 2, 0.3)])
def test_step_by_step_against_numerical_solve_of_eq2(d, g, r, G, bits, lam):
    # Replay the algorithm with the update of every step obtained from a plain least-squares solve
    # of Eq. (2) (no P_inv, no W): fixed coordinates stay, block t moves to its grid value, the
    # rest minimises ||delta||^2 + lam ||Qhat delta||^2.  Same final keys, same codes, and the same
    # error projected on the subspace.
    K, mats = _case(70 + d + g, G, d, r, lam, g, n_q=40, outliers=False)
    Qhat = mats["Qhat"]
    out = oracle.quant_keys(K, G, bits, mats["W"])
    L = 2 ** bits - 1
    S = np.vstack([np.eye(d), np.sqrt(lam) * Qhat])
    X = K.copy()
    codes = np.zeros((G, d), dtype=np.uint8)
    for t in range(1, d // g + 1):
        lo, hi = (t - 1) * g, t * g
        m, Mx = X[:, lo:hi].min(axis=0), X[:, lo:hi].max(axis=0)
        zf, sf = m.astype(np.float32).astype(np.float64), ((Mx - m) / L).astype(np.float32).astype(np.float64)
        c = np.clip(np.rint((X[:, lo:hi] - zf) / sf), 0, L)
        codes[:, lo:hi] = c
        xhat = zf + sf * c
        dvec = xhat - X[:, lo:hi]
        X[:, lo:hi] = xhat
        if hi < d:
            for i in range(G):
                z, *_ = np.linalg.lstsq(S[:, hi:], -S[:, lo:hi] @ dvec[i], rcond=None)
                X[i, hi:] += z
    assert np.array_equal(codes, out["codes"])
    assert np.allclose(X, out["Khat"], atol=1e-9)
    assert np.allclose((X - K) @ Qhat.T, (out["Khat"] - K) @ Qhat.T, atol=1e-8)


def test_exhaustive_search_cannot_be_beaten_from_below():
    # d = 6, b = 2: with the oracle's final grids held fixed, the global minimum of delta^T P delta
    # over all 4^6 code vectors is a lower bound for what the greedy algorithm reached, and the
    # greedy value stays within a small factor of it on this seeded case.
    d, G, bits, lam = 6, 4, 2, 0.5
    K, mats = _case(90, G, d, 2, lam, 1, n_q=30, outliers=False)
    out = oracle.quant_keys(K, G, bits, mats["W"])
    P = mats["P"]
    all_codes = np.array(list(itertools.product(range(4), repeat=d)), dtype=np.float64)
    sc, zr = out["scale"][0].astype(np.float64), out["zero"][0].astype(np.float64)
    grid = zr + sc * all_codes                                # [4^d, d]
    for i in range(G):
        dl = grid - K[i]
        obj = np.einsum("ij,jk,ik->i", dl, P, dl)
        mine = (out["Khat"][i] - K[i]) @ P @ (out["Khat"][i] - K[i])
        assert obj.min() <= mine + 1e-12
        assert mine <= 4.0 * obj.min() + 1e-12


def test_projected_error_is_below_round_to_nearest():
    # Section 3.3 / Figure 2: the residual is more orthogonal to the query subspace than with
    # compression-only quantization, at the price of a larger plain error.
    cfg = si.get_config(0)
    Qc = si.to_f32(si.gen_queries_head(cfg, 0), cfg.dtype).astype(np.float64)
    K = si.to_f32(si.gen_keys_unit(cfg, 0, 0), cfg.dtype).astype(np.float64)
    mats = oracle.build_W(Qc, cfg.rank_r, cfg.lam, 1)
    sq = oracle.quant_keys(K, cfg.group_size, cfg.bits, mats["W"])
    rt = oracle.quant_keys(K, cfg.group_size, cfg.bits, None)
    proj = lambda o: np.linalg.norm((o["Khat"] - K) @ mats["Qhat"].T)
    assert proj(sq) < 0.6 * proj(rt)
    assert np.linalg.norm(sq["Khat"] - K) > np.linalg.norm(rt["Khat"] - K)


def test_idempotent():
    K, mats = _case(5, 64, 64, 8, 0.01)
    a = oracle.quant_keys(K, 32, 2, mats["W"])
    b = oracle.quant_keys(a["Khat"], 32, 2, mats["W"])
    assert np.array_equal(a["codes"], b["codes"])
    assert np.array_equal(a["Khat"], b["Khat"])
    assert np.array_equal(a["scale"], b["scale"]) and np.array_equal(a["zero"], b["zero"])


def test_chunking_invariance():
    K, mats = _case(6, 128, 32, 4, 0.05)
    whole = oracle.quant_keys(K, 32, 2, mats["W"])
    for lo, hi in [(0, 32), (32, 96), (96, 128)]:
        part = oracle.quant_keys(K[lo:hi], 32, 2, mats["W"])
        assert np.array_equal(part["codes"], whole["codes"][lo:hi])
        assert np.array_equal(part["scale"], whole["scale"][lo // 32:hi // 32])
        assert np.array_equal(part["Khat"], whole["Khat"][lo:hi])


def test_constant_group_has_zero_scale():
    K, mats = _case(7, 32, 16, 2, 0.05)
    K[:, 3] = 1.25
    mats["W"][:, :] = 0.0
    out = oracle.quant_keys(K, 32, 2, mats["W"])
    assert out["scale"][0, 3] == 0.0 and out["zero"][0, 3] == np.float32(1.25)
    assert not out["codes"][:, 3].any()
    assert np.array_equal(out["Khat"][:, 3], K[:, 3])


def test_forced_code_is_used_and_propagates():
    K, mats = _case(8, 32, 16, 3, 0.5)
    base = oracle.quant_keys(K, 32, 2, mats["W"], want_tval=True)
    force = -np.ones((32, 16), dtype=np.int16)
    i, j = 5, 2
    alt = (int(base["codes"][i, j]) + 1) % 4
    force[i, j] = alt
    out = oracle.quant_keys(K, 32, 2, mats["W"], force=force)
    assert out["codes"][i, j] == alt
    assert np.array_equal(out["codes"][:, :j], base["codes"][:, :j])
    assert np.isclose(out["Khat"][i, j], out["zero"][0, j] + out["scale"][0, j] * np.float64(alt))
    # the other tokens of the group are untouched up to the point where channel grids change
    assert not np.allclose(out["Khat"][i, j + 1:], base["Khat"][i, j + 1:])
    # tval reports (x - zero)/scale: rounding it reproduces the codes
    assert np.array_equal(np.clip(np.rint(base["tval"]), 0, 3).astype(np.uint8), base["codes"])
