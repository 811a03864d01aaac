"""GPU parity of the projected FIM, its damped Cholesky solve and the preconditioned score."""
import numpy as np
import pytest
import torch

from parity import check_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import paper_2505_18976_b200 as g
    g.lib()
    return g


def _compressed(n, k, seed, scale=1.0):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    # correlated columns so that F is far from a multiple of the identity
    Z = torch.randn((n, k), generator=g, device="cuda")
    mix = torch.randn((k, k), generator=g, device="cuda") / k ** 0.5
    return ((Z + 0.5 * Z @ mix) * scale).contiguous()


@pytest.mark.parametrize("n,k", [(1000, 96), (77, 130), (4096, 256), (33, 1), (3000, 520)])
def test_fim_parity(G, oracle_mod, n, k):
    X = _compressed(n, k, 3 + k)
    F = G.grass_fim(X).cpu().numpy()
    ref, absum = oracle_mod.fim(X.cpu().numpy())
    check_close(F, ref, absum, 1e-4, n + 64, eps=2.0 ** -23, what=f"fim n={n} k={k}")
    # mirrored entries get the same addends, possibly in another order across sample chunks
    assert np.all(np.abs(F - F.T) <= 2.0 ** -21 * absum)


def test_fim_of_a_column_slice(G, oracle_mod):
    """One layer's block of a wider compressed matrix (block-diagonal FIM)."""
    X = _compressed(500, 300, 9)
    blk = X[:, 100:228]
    F = G.grass_fim(blk).cpu().numpy()
    ref, absum = oracle_mod.fim(np.ascontiguousarray(blk.cpu().numpy()))
    check_close(F, ref, absum, 1e-4, 564, eps=2.0 ** -23, what="fim column slice")


@pytest.mark.parametrize("n,k,lam,M", [(600, 64, 1e-2, 5), (900, 200, 1e-1, 70), (2000, 333, 1e-2, 256), (50, 100, 0.5, 3)])
def test_factor_and_apply_parity(G, oracle_mod, n, k, lam, M):
    X = _compressed(n, k, 20 + k)
    B = _compressed(M, k, 21 + k)
    F = G.grass_fim(X)
    Fh = F.cpu().numpy().astype(np.float64)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    L = G.grass_fim_factor(F.clone(), lam, dev_status=st)
    sol = G.grass_fim_apply(L, B.clone()).cpu().numpy().astype(np.float64)
    assert int(st.item()) == 0
    # the factor itself: L L^T = F + lam I
    Lh = np.tril(L.cpu().numpy().astype(np.float64))
    Mh = Fh + lam * np.eye(k)
    assert np.abs(Lh @ Lh.T - Mh).max() <= 1e-5 * np.abs(Mh).max()
    # the solution against the oracle on the same matrix, within the conditioning of the system
    ref = oracle_mod.fim_solve(Fh, lam, B.cpu().numpy().astype(np.float64))
    cond = np.linalg.cond(Mh)
    err = np.linalg.norm(sol - ref, axis=1) / np.linalg.norm(ref, axis=1)
    assert err.max() <= 64 * cond * 2.0 ** -24, (err.max(), cond)
    # and against the oracle chain from the raw data (fim in double, then solve)
    ref2 = oracle_mod.fim_solve(oracle_mod.fim(X.cpu().numpy())[0], lam, B.cpu().numpy().astype(np.float64))
    err2 = np.linalg.norm(sol - ref2, axis=1) / np.linalg.norm(ref2, axis=1)
    assert err2.max() <= 64 * cond * 2.0 ** -23


def test_not_positive_definite_is_flagged(G):
    F = torch.zeros(70, 70, device="cuda")
    F[0, 0] = -1.0
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    G.grass_fim_factor(F, 0.0, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == G.binding.DEV_NOT_PD


def test_preconditioned_score(G, oracle_mod):
    """scores[i, m] = <g_i, (F + lam I)^-1 g_test,m> through grass_fim -> factor -> apply -> grass_score."""
    n, k, M, lam = 1500, 192, 40, 5e-2
    train = _compressed(n, k, 50)
    test = _compressed(M, k, 51)
    L = G.grass_fim_factor(G.grass_fim(train), lam)
    pt = G.grass_fim_apply(L, test.clone())
    sc = G.grass_score(train, pt).cpu().numpy().astype(np.float64)
    th, eh = train.cpu().numpy(), test.cpu().numpy()
    ref = th.astype(np.float64) @ oracle_mod.fim_solve(oracle_mod.fim(th)[0], lam, eh.astype(np.float64)).T
    cond = np.linalg.cond(oracle_mod.fim(th)[0] + lam * np.eye(k))
    scale = np.linalg.norm(ref, axis=0, keepdims=True) / np.sqrt(n)
    assert (np.abs(sc - ref) / scale).max() <= 64 * cond * 2.0 ** -23
