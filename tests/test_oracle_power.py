"""Pins of the oracle's block power method (the accelerator named for line 5 of Algorithm 1) against what the
mathematics fixes: the span after q steps is that of M^q X0 (checked through an explicit matrix power and an
SVD-based projector), closed forms for diagonal M, exactness when rank(M) <= r, geometric convergence to the exact
rank-r truncation when there is a gap, invariance under a change of basis of the start block, and Cauchy
interlacing of the Ritz values."""
import numpy as np
import pytest

import oracle
import squat_inputs as si


def _sym_with_spectrum(mu, seed):
    d = len(mu)
    rng = np.random.default_rng(seed)
    V, _ = np.linalg.qr(rng.standard_normal((d, d)))
    return (V * np.asarray(mu, dtype=np.float64)) @ V.T, V


def test_span_is_that_of_the_matrix_power_applied_to_the_start_block():
    d, r = 24, 5
    M, _ = _sym_with_spectrum(np.linspace(3.0, 1.0, d), 1)
    X0 = si.gen_start_block(11, d, r)
    for q in (0, 1, 2, 3):
        Qhat, theta, X = oracle.power_subspace(M, X0, q)
        Z = np.linalg.matrix_power(M, q) @ X0
        U, s, _ = np.linalg.svd(Z, full_matrices=False)          # independent route to the projector
        Pi = U @ U.T
        assert np.abs(X @ X.T - Pi).max() < 1e-10
        assert np.abs(Qhat.T @ Qhat - Pi @ M @ Pi).max() < 1e-10 * np.abs(M).max() * 10
        assert np.all(np.diff(theta) <= 1e-12)
        G = Qhat @ Qhat.T                                        # rows orthogonal, squared norms = Ritz values
        assert np.abs(G - np.diag(theta)).max() < 1e-10


def test_diagonal_matrix_and_coordinate_start_block_closed_form():
    d, lam = 16, 0.37
    mu = np.array([5.0, 0.5, 7.0, 1.0, 3.0, 0.25, 9.0, 2.0, 4.0, 6.0, 8.0, 0.75, 1.5, 2.5, 3.5, 4.5])
    J = [2, 6, 9, 12]                                             # the span never leaves these coordinates
    X0 = np.zeros((d, len(J)))
    for c, j in enumerate(J):
        X0[j, c] = 1.0 + 0.1 * c
    X0[:, 1] += X0[:, 0]                                          # a non-orthogonal basis of the same span
    for q in (0, 1, 4):
        Qhat, theta, _ = oracle.power_subspace(np.diag(mu), X0, q)
        assert np.allclose(theta, sorted(mu[J], reverse=True), rtol=1e-12)
        mats = oracle.update_matrices(Qhat, d, lam)
        expect = np.ones(d)
        expect[J] += lam * mu[J]
        assert np.abs(mats["P"] - np.diag(expect)).max() < 1e-12
        assert np.abs(mats["W"]).max() < 1e-12                    # diagonal P: no error feedback at all


@pytest.mark.parametrize("k", [3, 8])
def test_exact_after_one_step_when_the_rank_fits_the_block(k):
    d, r, lam = 32, 8, 0.05
    rng = np.random.default_rng(3)
    Qc = rng.standard_normal((k, d)) * 3.0                        # rank k <= r
    exact = oracle.build_W(Qc, r, lam)
    X0 = si.gen_start_block(5, d, r)
    got = oracle.build_W_power(Qc, X0, 1, lam)
    assert np.abs(got["P"] - exact["P"]).max() < 1e-10 * np.abs(exact["P"]).max()
    assert np.abs(got["W"] - exact["W"]).max() < 1e-10
    assert np.abs(got["theta"][:k] - exact["mu"][:k]).max() < 1e-10 * exact["mu"][0]
    assert np.abs(got["theta"][k:]).max(initial=0.0) < 1e-10 * exact["mu"][0]


def test_converges_geometrically_to_the_rank_r_truncation_when_there_is_a_gap():
    d, r, lam = 40, 6, 0.2
    mu = np.concatenate([np.linspace(10.0, 5.0, r), np.linspace(0.05, 0.01, d - r)])   # gap 100 after r
    M, V = _sym_with_spectrum(mu, 7)
    P_exact = np.eye(d) + lam * (V[:, :r] * mu[:r]) @ V[:, :r].T
    X0 = si.gen_start_block(9, d, r)
    errs = []
    for q in range(0, 5):
        Qhat, _, _ = oracle.power_subspace(M, X0, q)
        errs.append(np.abs(np.eye(d) + lam * Qhat.T @ Qhat - P_exact).max())
    assert errs[0] > 0.1
    for q in range(1, 4):
        assert errs[q] < errs[q - 1] * 0.05                       # the angle shrinks by mu_{r+1}/mu_r = 0.01 per step
    assert errs[4] < 1e-7


def test_result_depends_on_the_span_of_the_start_block_only():
    cfg = si.get_config(0)
    Qc = si.to_f32(si.gen_queries_head(cfg, 0, 256), cfg.dtype).astype(np.float64)
    d, r = Qc.shape[1], 8
    X0 = si.gen_start_block(cfg.seed, d, r)
    A = np.random.default_rng(2).standard_normal((r, r)) + 3.0 * np.eye(r)
    a = oracle.build_W_power(Qc, X0, 2, cfg.lam)
    b = oracle.build_W_power(Qc, X0 @ A, 2, cfg.lam)
    assert np.abs(a["W"] - b["W"]).max() < 1e-10
    assert np.abs(a["P"] - b["P"]).max() < 1e-10 * np.abs(a["P"]).max()


def test_ritz_values_interlace_the_eigenvalues():
    cfg = si.get_config(0)
    Qc = si.to_f32(si.gen_queries_head(cfg, 1, 300), cfg.dtype).astype(np.float64)
    d, r = Qc.shape[1], 12
    M = oracle.gram(Qc)
    mu = np.linalg.eigvalsh(M)[::-1]
    prev = None
    for q in (0, 1, 2, 3):
        _, theta, _ = oracle.power_subspace(M, si.gen_start_block(4, d, r), q)
        assert np.all(theta <= mu[:r] * (1 + 1e-12))              # Cauchy interlacing, upper side
        assert np.all(theta >= mu[d - r:] * (1 - 1e-12))          # and lower side
        if prev is not None:
            assert theta.sum() >= prev - 1e-9 * mu[0]             # power steps only add captured energy
        prev = theta.sum()


def test_on_the_workload_generator_two_steps_capture_the_signal_directions():
    # config 1's queries: 16 strong directions, a flat noise floor below; r = 32 cuts inside the floor, where the
    # power method and the SVD pick different (equally small) directions: P agrees to 1e-3, the captured query energy
    # to 1e-4, and the signal eigenvalues to 1e-8
    cfg = si.get_config(1)
    Qc = si.to_f32(si.gen_queries_head(cfg, 0, 1024), cfg.dtype).astype(np.float64)
    d, r = Qc.shape[1], cfg.rank_r
    M = oracle.gram(Qc)
    mu, V = np.linalg.eigh(M)
    mu, V = mu[::-1], V[:, ::-1]
    Qhat, theta, _ = oracle.power_subspace(M, si.gen_start_block(cfg.seed, d, r), 2)
    P_exact = np.eye(d) + cfg.lam * (V[:, :r] * mu[:r]) @ V[:, :r].T
    P = np.eye(d) + cfg.lam * Qhat.T @ Qhat
    assert np.linalg.norm(P - P_exact) < 1e-3 * np.linalg.norm(P_exact)
    assert abs(theta.sum() / mu[:r].sum() - 1.0) < 1e-4
    assert np.abs(theta[:16] / mu[:16] - 1.0).max() < 1e-8
