"""Pins of the oracle's projected Fisher information matrix and damped iFVP (CPU only):
closed forms, numpy's own factorisation, the residual of the linear system, and the
preconditioned score assembled from pinned parts."""
import numpy as np
import pytest


def test_fim_is_the_averaged_outer_product(oracle_mod):
    rng = np.random.default_rng(1)
    X = rng.standard_normal((37, 9)).astype(np.float32)
    F, ab = oracle_mod.fim(X)
    Xd = X.astype(np.float64)
    ref = sum(np.outer(Xd[i], Xd[i]) for i in range(37)) / 37            # the definition, sample by sample
    np.testing.assert_allclose(F, ref, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(ab, np.abs(Xd).T @ np.abs(Xd) / 37, rtol=1e-13)
    assert np.array_equal(F, F.T)
    assert np.linalg.eigvalsh(F).min() > -1e-12                           # positive semi-definite
    # one sample: rank one, F = g g^T
    F1, _ = oracle_mod.fim(X[:1])
    np.testing.assert_allclose(F1, np.outer(Xd[0], Xd[0]), rtol=1e-15)
    # orthogonal one-hot samples: diagonal matrix of counts / n
    E = np.zeros((6, 4), dtype=np.float32)
    E[[0, 1, 2, 3, 4, 5], [0, 0, 1, 3, 3, 3]] = 2.0
    Fe, _ = oracle_mod.fim(E)
    np.testing.assert_array_equal(Fe, np.diag([2, 1, 0, 3]) * 4.0 / 6)


def test_solve_closed_forms(oracle_mod):
    # diagonal F: x = b / (f + lambda)
    f = np.array([4.0, 1.0, 0.0, 9.0])
    b = np.array([[1.0, 2.0, 3.0, 4.0], [0.0, -1.0, 5.0, 2.0]])
    x = oracle_mod.fim_solve(np.diag(f), 0.5, b)
    np.testing.assert_allclose(x, b / (f + 0.5), rtol=1e-15)
    # F = 0: x = b / lambda
    np.testing.assert_allclose(oracle_mod.fim_solve(np.zeros((4, 4)), 0.25, b), b * 4, rtol=1e-15)
    # rank-one F = u u^T (Sherman-Morrison): (uu^T + l I)^-1 b = (b - u (u.b) / (l + u.u)) / l
    u = np.array([1.0, -2.0, 0.5, 3.0])
    lam = 0.7
    ref = (b - np.outer(b @ u, u) / (lam + u @ u)) / lam
    np.testing.assert_allclose(oracle_mod.fim_solve(np.outer(u, u), lam, b), ref, rtol=1e-13)
    # not positive definite without damping
    with pytest.raises(np.linalg.LinAlgError):
        oracle_mod.fim_solve(np.outer(u, u), 0.0, b)


@pytest.mark.parametrize("k,n,lam", [(12, 40, 1e-3), (50, 20, 1e-2), (33, 200, 0.0)])
def test_solve_against_numpy_and_residual(oracle_mod, k, n, lam):
    rng = np.random.default_rng(k)
    X = rng.standard_normal((n, k)).astype(np.float32)
    F, _ = oracle_mod.fim(X)
    B = rng.standard_normal((7, k))
    x = oracle_mod.fim_solve(F, lam, B)
    M = F + lam * np.eye(k)
    np.testing.assert_allclose(x, np.linalg.solve(M, B.T).T, rtol=1e-8, atol=1e-10)
    np.testing.assert_allclose(x @ M, B, rtol=1e-8, atol=1e-9)            # residual of the system itself
    # a transposed or unsymmetrised factor would break this: solve with M^T = M gives the same
    np.testing.assert_allclose(oracle_mod.fim_solve(F.T.copy(), lam, B), x, rtol=1e-12)


def test_preconditioned_score_is_symmetric_in_train_and_test(oracle_mod):
    """<g_test, F^-1 g_i> = <F^-1 g_test, g_i> (Section 2.1): preconditioning either side gives the same scores."""
    rng = np.random.default_rng(5)
    k = 20
    train = rng.standard_normal((30, k)).astype(np.float32)
    test = rng.standard_normal((4, k)).astype(np.float32)
    F, _ = oracle_mod.fim(train)
    lam = 1e-2
    pt = oracle_mod.fim_solve(F, lam, test.astype(np.float64))
    ptr = oracle_mod.fim_solve(F, lam, train.astype(np.float64))
    a = train.astype(np.float64) @ pt.T
    b = ptr @ test.astype(np.float64).T
    np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-11)
    # self-influence is positive: g^T (F + l I)^-1 g > 0
    assert np.all(np.einsum("ik,ik->i", train.astype(np.float64), ptr) > 0)
