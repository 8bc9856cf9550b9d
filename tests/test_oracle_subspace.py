"""Pins of the oracle's projection step (Algorithm 2, the SVD lines): the top-r
left singular subspace by definition, and the randomised subspace iteration the
GPU follows, against closed-form cases and each other."""
import numpy as np
import pytest

from oracle import loqt_oracle as O


def _lowrank(seed, out, inn, r, decay=0.5, noise=1e-3):
    """G = U diag(s) V^T + noise with known orthonormal U: the top-r subspace is span(U[:, :r])."""
    rng = np.random.default_rng(seed)
    U, _ = np.linalg.qr(rng.normal(size=(out, min(out, inn))))
    V, _ = np.linalg.qr(rng.normal(size=(inn, min(out, inn))))
    k = min(out, inn)
    s = np.concatenate([np.linspace(2.0, 1.0, r), decay * np.linspace(1.0, 0.1, k - r)])
    return (U * s) @ V.T + noise * rng.normal(size=(out, inn)), U[:, :r], s


def test_definition_recovers_a_planted_subspace_and_is_orthonormal():
    G, U_r, _ = _lowrank(0, 96, 160, 12, decay=0.3, noise=0.0)
    P = O.top_r_left_subspace(G, 12)
    assert np.allclose(P.T @ P, np.eye(12), atol=1e-12)
    assert np.max(O.subspace_sines(U_r, P)) < 1e-10
    # it is the best rank-r projection: the captured energy equals the sum of the r largest squared singular values
    sv = np.linalg.svd(G, compute_uv=False)
    assert np.isclose(np.linalg.norm(P.T @ G) ** 2, np.sum(sv[:12] ** 2), rtol=1e-12)
    # a diagonal matrix: the subspace is spanned by the unit vectors of its largest entries
    D = np.diag([5.0, 0.1, 3.0, 0.2, 4.0, 0.3])
    Pd = O.top_r_left_subspace(D, 3)
    assert np.allclose(np.abs(Pd).sum(axis=1), [1, 0, 1, 0, 1, 0], atol=1e-12)


def test_principal_angle_helper():
    e = np.eye(4)
    assert np.allclose(O.subspace_sines(e[:, :2], e[:, :2]), 0)
    assert np.allclose(O.subspace_sines(e[:, :2], e[:, 2:]), 1)
    c, s = np.cos(0.3), np.sin(0.3)
    Q = np.stack([c * e[:, 0] + s * e[:, 2], e[:, 1]], axis=1)
    assert np.allclose(sorted(O.subspace_sines(e[:, :2], Q)), [0, s], atol=1e-12)


@pytest.mark.parametrize("shape", [(96, 160, 12), (200, 120, 24)])
def test_iteration_is_exact_for_exact_rank_and_converges_at_the_gap_rate(shape):
    out, inn, r = shape
    rng = np.random.default_rng(1)
    Omega = rng.normal(size=(inn, r))
    # exact rank r: one multiplication already spans the column space
    G0, U_r, _ = _lowrank(2, out, inn, r, decay=0.0, noise=0.0)
    Q = O.subspace_iteration(G0, Omega, 0)
    assert np.allclose(Q.T @ Q, np.eye(r), atol=1e-12)
    assert np.max(O.subspace_sines(U_r, Q)) < 1e-9
    # a spectral gap of 1/2: the error shrinks by about (1/2)^2 per iteration
    G, _, s = _lowrank(3, out, inn, r, decay=0.5, noise=0.0)
    P = O.top_r_left_subspace(G, r)
    err = [np.max(O.subspace_sines(P, O.subspace_iteration(G, Omega, q))) for q in range(6)]
    assert all(err[q + 1] < err[q] for q in range(5))
    # once the iterate is near the subspace, (sigma_{r+1} / sigma_r)^2 = 1/4 per iteration
    assert all(err[q + 1] < 0.3 * err[q] for q in range(1, 5))
    assert err[5] < 3e-3
    # the captured energy approaches the optimum from below
    opt = np.linalg.norm(P.T @ G) ** 2
    cap = [np.linalg.norm(O.subspace_iteration(G, Omega, q).T @ G) ** 2 for q in (0, 1, 3)]
    assert cap[0] <= cap[1] <= cap[2] <= opt * (1 + 1e-12) and cap[2] > 0.999 * opt


def test_iteration_matches_plain_power_iteration_for_rank_one():
    # r = 1: subspace iteration is the power method on G G^T
    rng = np.random.default_rng(4)
    G = rng.normal(size=(30, 50))
    w = rng.normal(size=(50, 1))
    y = G @ w
    for _ in range(3):
        y = G @ (G.T @ (y / np.linalg.norm(y)))
    y /= np.linalg.norm(y)
    Q = O.subspace_iteration(G, w, 3)
    assert min(np.linalg.norm(Q - y), np.linalg.norm(Q + y)) < 1e-10


def test_right_side_recovers_a_planted_right_subspace():
    # G = U diag(s) V^T with known V: the top-r right subspace is span(V[:, :r]); the iteration converges to it
    out, inn, r = 160, 96, 12
    rng = np.random.default_rng(5)
    U, _ = np.linalg.qr(rng.normal(size=(out, inn)))
    V, _ = np.linalg.qr(rng.normal(size=(inn, inn)))
    s = np.concatenate([np.linspace(2.0, 1.0, r), 0.3 * np.linspace(1.0, 0.1, inn - r)])
    G = (U * s) @ V.T
    Qd = O.top_r_right_subspace(G, r)
    assert Qd.shape == (r, inn) and np.allclose(Qd @ Qd.T, np.eye(r), atol=1e-12)
    assert np.max(O.subspace_sines(V[:, :r], Qd.T)) < 1e-10
    # what the right-side variant needs of it: G Q^T Q keeps the energy of the r largest singular values
    assert np.isclose(np.linalg.norm(G @ Qd.T) ** 2, np.sum(s[:r] ** 2), rtol=1e-12)
    Omega = rng.normal(size=(out, r))
    err = [np.max(O.subspace_sines(V[:, :r], O.subspace_iteration_right(G, Omega, q).T)) for q in range(5)]
    assert all(err[q + 1] < 0.3 * err[q] for q in range(1, 4)) and err[4] < 1e-3
    Q = O.subspace_iteration_right(G, Omega, 2)
    assert Q.shape == (r, inn) and np.allclose(Q @ Q.T, np.eye(r), atol=1e-12)
