"""Pins for the oracle's update matrices (Prop. 1, Prop. 2, Lemma 3, Lemma 4).

Nothing here calls the CUDA library.  Every check compares the oracle with something
that is not the oracle: a library inverse, a generic least-squares solve of the
optimisation problem the paper derives the update from, or a library Cholesky factor.
"""
import numpy as np
import pytest

import oracle


def _random_qhat(rng, r, d, scale=3.0):
    return scale * rng.standard_normal((r, d))


@pytest.mark.parametrize("d,g", [(16, 1), (16, 2), (16, 4), (16, 8), (24, 3), (12, 12), (128, 1), (128, 32), (128, 64)])
def test_chain_equals_direct_inverse(d, g):
    # Lemma 4 / Prop. 2: A_t^{-1} from the downdate chain equals inverse(top-left tg x tg of P_inv).
    rng = np.random.default_rng(10 + d + g)
    Qhat = _random_qhat(rng, min(5, d), d)
    m = oracle.update_matrices(Qhat, d, 0.05, g, want_chain=True)
    P_np = np.eye(d) + 0.05 * Qhat.T @ Qhat
    assert np.allclose(m["P"], P_np, rtol=0, atol=1e-12)
    Pinv_np = np.linalg.inv(P_np)
    assert np.abs(m["P_inv"] - Pinv_np).max() < 1e-12
    T = d // g
    ts = range(1, T + 1) if d <= 24 else sorted({1, 2, T // 2, T - 1, T} & set(range(1, T + 1)))
    for t in ts:
        direct = np.linalg.inv(Pinv_np[: t * g, : t * g])
        rel = np.abs(m["Ainv"][t] - direct).max() / np.abs(direct).max()
        assert rel < 1e-10, (t, rel)


@pytest.mark.parametrize("d,g,r", [(16, 1, 3), (16, 4, 5), (24, 2, 24), (128, 1, 32), (128, 32, 8)])
def test_update_equals_schur_solve(d, g, r):
    # U_t = B_t H_t equals -P22^{-1} P21 restricted to block t's columns
    # (minimiser of delta^T P delta with the head of delta fixed; Lemma 1 applied to P).
    rng = np.random.default_rng(20 + d + g)
    Qhat = _random_qhat(rng, r, d)
    lam = 0.02
    W = oracle.update_matrices(Qhat, d, lam, g)["W"]
    P = np.eye(d) + lam * Qhat.T @ Qhat
    for t in range(1, d // g):
        lo, hi = (t - 1) * g, t * g
        U = -np.linalg.solve(P[hi:, hi:], P[hi:, lo:hi])
        assert np.abs(W[hi:, lo:hi] - U).max() < 1e-11
        # nothing on or above the block diagonal
        assert not W[:hi, lo:hi].any()
    assert not W[:, d - g:].any()


@pytest.mark.parametrize("d,g,r,lam", [(8, 1, 3, 0.3), (8, 2, 2, 1.0), (12, 4, 5, 0.01), (6, 3, 1, 10.0)])
def test_update_solves_the_papers_problem(d, g, r, lam):
    # Lemma 3, Eq. (gen_upd_opt): minimise ||delta||^2 + lam ||Qhat delta||^2 subject to
    # delta = 0 on the first (t-1)g coordinates and delta = dvec on block t.  Solve it as a plain
    # linear least-squares problem in the free coordinates (no P_inv, no closed form) and compare.
    rng = np.random.default_rng(30 + d + g)
    Qhat = _random_qhat(rng, r, d, scale=1.5)
    W = oracle.update_matrices(Qhat, d, lam, g)["W"]
    S = np.vstack([np.eye(d), np.sqrt(lam) * Qhat])      # objective = ||S delta||^2
    for t in range(1, d // g):
        lo, hi = (t - 1) * g, t * g
        dvec = rng.standard_normal(g)
        z, *_ = np.linalg.lstsq(S[:, hi:], -S[:, lo:hi] @ dvec, rcond=None)
        assert np.abs(W[hi:, lo:hi] @ dvec - z).max() < 1e-10


def test_elementwise_is_block_case_with_g1():
    # Prop. 1 written out: last d-t elements move by d * B_t h_t, h_t = last column of A_t^{-1}.
    rng = np.random.default_rng(41)
    d, lam = 10, 0.2
    Qhat = _random_qhat(rng, 4, d)
    W = oracle.update_matrices(Qhat, d, lam, 1)["W"]
    Pinv = np.linalg.inv(np.eye(d) + lam * Qhat.T @ Qhat)
    for t in range(1, d):
        h_t = np.linalg.inv(Pinv[:t, :t])[:, -1]
        assert np.abs(W[t:, t - 1] - Pinv[t:, :t] @ h_t).max() < 1e-12


@pytest.mark.parametrize("d", [8, 32, 128])
def test_unit_lower_ldl_factor(d):
    # g = 1: I + W is the unit-lower factor of P_inv = (I+W) D (I+W)^T.
    rng = np.random.default_rng(50 + d)
    Qhat = _random_qhat(rng, 6, d)
    lam = 0.05
    W = oracle.update_matrices(Qhat, d, lam, 1)["W"]
    C = np.linalg.cholesky(np.linalg.inv(np.eye(d) + lam * Qhat.T @ Qhat))
    Lunit = C / np.diag(C)[None, :]
    assert np.abs(np.eye(d) + W - Lunit).max() < 1e-11


def test_no_subspace_means_no_update():
    # lambda = 0 (or r = 0): P = I and the method reduces to plain compression (Section 3.3).
    rng = np.random.default_rng(60)
    d = 16
    Qhat = _random_qhat(rng, 4, d)
    assert not oracle.update_matrices(Qhat, d, 0.0, 1)["W"].any()
    assert not oracle.update_matrices(np.zeros((0, d)), d, 1e-3, 4)["W"].any()


def test_bad_arguments_are_rejected():
    with pytest.raises(RuntimeError):
        oracle.update_matrices(np.zeros((1, 8)), 8, 1e-3, 3)      # g does not divide d
    with pytest.raises(RuntimeError):
        oracle.update_matrices(np.zeros((1, 8)), 8, -1.0, 1)      # negative lambda
