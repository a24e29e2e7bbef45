"""Pins for the oracle's LAPACK-free SVD routines."""
import numpy as np
import pytest

from oracle import lqer


def _check_svd(G, U, s, Vt, tol=1e-12):
    r = min(G.shape)
    assert U.shape == (G.shape[0], r) and s.shape == (r,) and Vt.shape == (r, G.shape[1])
    assert np.all(np.diff(s) <= 1e-15 * max(1.0, s[0])) and np.all(s >= 0)
    assert np.abs(U.T @ U - np.eye(r)).max() <= tol
    assert np.abs(Vt @ Vt.T - np.eye(r)).max() <= tol
    assert np.abs((U * s) @ Vt - G).max() <= tol * max(1.0, np.abs(G).max()) * max(G.shape)


@pytest.mark.parametrize("shape", [(7, 7), (40, 24), (24, 40), (96, 64), (33, 17)])
def test_random_matrices(shape):
    g = np.random.default_rng(shape[0] * 100 + shape[1])
    G = g.standard_normal(shape)
    U, s, Vt = lqer.jacobi_svd(G)
    _check_svd(G, U, s, Vt)
    # singular values squared are the eigenvalues of the Gram matrix: trace and determinant pins
    assert np.isclose(np.sum(s ** 2), np.sum(G * G), rtol=1e-12)


def test_diagonal_closed_form():
    d = np.array([3.0, -7.0, 0.5, 2.0])
    U, s, Vt = lqer.jacobi_svd(np.diag(d))
    assert np.allclose(s, [7.0, 3.0, 2.0, 0.5], rtol=0, atol=1e-15)
    _check_svd(np.diag(d), U, s, Vt)


def test_rank_one_closed_form():
    u = np.array([1.0, 2.0, -2.0])          # |u| = 3
    v = np.array([3.0, 0.0, 4.0, 0.0])      # |v| = 5
    G = np.outer(u, v)
    U, s, Vt = lqer.jacobi_svd(G)
    assert np.isclose(s[0], 15.0, rtol=1e-14) and np.all(s[1:] < 1e-13)
    assert np.allclose(np.abs(U[:, 0]), np.abs(u) / 3.0, atol=1e-14)
    assert np.allclose(np.abs(Vt[0]), np.abs(v) / 5.0, atol=1e-14)
    assert np.abs(U.T @ U - np.eye(3)).max() < 1e-12


def test_two_by_two_closed_form():
    # singular values of [[a, b], [c, d]]: sqrt((q +- sqrt(q^2 - 4 det^2)) / 2), q = a^2+b^2+c^2+d^2
    a, b, c, d = 3.0, 1.0, -2.0, 4.0
    q = a * a + b * b + c * c + d * d
    det = a * d - b * c
    root = np.sqrt(q * q - 4 * det * det)
    want = np.sqrt(np.array([(q + root) / 2, (q - root) / 2]))
    _, s, _ = lqer.jacobi_svd(np.array([[a, b], [c, d]]))
    assert np.allclose(s, want, rtol=1e-14)


def test_orthogonal_input_has_unit_spectrum():
    g = np.random.default_rng(3)
    Q = lqer._orthonormalise(g.standard_normal((20, 20)))
    _, s, _ = lqer.jacobi_svd(Q)
    assert np.allclose(s, 1.0, atol=1e-12)


def test_subspace_iteration_matches_jacobi_on_decaying_spectrum():
    g = np.random.default_rng(11)
    m, n, k = 160, 224, 12
    U = lqer._orthonormalise(g.standard_normal((m, m)))
    V = lqer._orthonormalise(g.standard_normal((n, m)))
    sig = np.concatenate([np.linspace(10, 4, k), 0.5 * np.exp(-0.05 * np.arange(m - k))])
    G = (U * sig) @ V.T
    Uj, sj, Vtj = lqer.jacobi_svd(G)
    assert np.allclose(sj, np.sort(sig)[::-1], rtol=1e-10)
    Us, ss, Vts = lqer.subspace_svd(G, k, np.random.default_rng(0))
    assert np.allclose(ss, sj[:k], rtol=1e-6)
    # same rank-k approximation (the factors may differ in sign)
    assert np.abs((Us * ss) @ Vts - (Uj[:, :k] * sj[:k]) @ Vtj[:k]).max() < 1e-5
