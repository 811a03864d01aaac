"""Accuracy of the fp32 contractions that run on bf16 tensor cores (grass_score, fp32-input FactGraSS / factorised
Mask, grass_fim): fp32 operands are split into bf16 pieces and the product is rebuilt from partial products.
The parity rule of tests/parity.py cannot see a missing correction term where sums cancel, so these tests use
operands of one sign (nothing cancels, every output is well conditioned) and bound the relative error directly,
against the oracle's fp64 values:

    all six partial products, D (T, n) = 512:   <= 4e-6   (truncating accumulators alone: 32 MMAs * 2^-24 ~ 2e-6;
                                                           a missing 2^-16 term with biased pieces would give ~1e-5)
    single accumulator over 4,096 k-values:      max|err| / max|ref| <= 2e-5 on signed data
"""
import numpy as np
import pytest
import torch

from parity import assert_accurate, check_close

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def G():
    import paper_2505_18976_b200 as g
    g.lib()
    return g


@pytest.fixture(scope="module")
def W():
    from paper_2505_18976_b200 import workloads
    return workloads


def _positive(shape, seed):
    g = torch.Generator(device="cuda")
    g.manual_seed(seed)
    return torch.rand(shape, generator=g, device="cuda") + 0.5          # [0.5, 1.5): full 24-bit mantissas


def _max_rel(gpu, ref):
    gpu = np.asarray(gpu, dtype=np.float64)
    return float((np.abs(gpu - ref) / np.abs(ref)).max())


def test_score_positive_operands_pin_all_six_products(G, oracle_mod, tune):
    tr, te = _positive((300, 512), 1), _positive((70, 512), 2)
    ref, _ = oracle_mod.score(tr.cpu().numpy(), te.cpu().numpy())
    tune(score_splits=1)
    rel = _max_rel(G.grass_score(tr, te).cpu().numpy(), ref)
    assert rel <= 4e-6, rel
    # the plain FMA kernel is the same arithmetic in IEEE fp32
    tune(score_ffma=1)
    assert _max_rel(G.grass_score(tr, te).cpu().numpy(), ref) <= 4e-6


@pytest.mark.parametrize("D", [4096, 8192])
def test_score_single_accumulator_accuracy(G, W, oracle_mod, tune, D):
    """The launch shape the benchmark times (one accumulator over the whole contraction) on signed data."""
    tune(score_splits=1)
    tr, te = W.score_vectors(384, 256, D, 5, device="cuda")
    sc = G.grass_score(tr, te).cpu().numpy()
    ref, absum = oracle_mod.score(tr.cpu().numpy(), te.cpu().numpy())
    # `rel` covers outputs down to |ref| = 2^-10 absum, where a sum of D signed terms has lost two to three
    # digits to cancellation: it is bounded loosely here, the arithmetic itself by assert_accurate
    rel = check_close(sc, ref, absum, 1e-4, D + 8, what=f"score D={D}, one accumulator")
    assert rel <= 1e-3
    assert_accurate(sc, ref, 2e-5, what=f"score D={D}, one accumulator")


def test_factmask_fp32_positive_operands(G, W, oracle_mod):
    """The k'_in x k'_out block of Eq. 2 from fp32 factors of one sign, T = 512, both tile sizes of the kernel."""
    B, T, d_in, d_out, kin, kout = 2, 512, 300, 200, 128, 70
    A, Gt = _positive((B, T, d_in), 3), _positive((B, T, d_out), 4)
    mi, mo = oracle_mod.random_mask(d_in, kin, 1), oracle_mod.random_mask(d_out, kout, 2)
    out = G.factmask_compress(A, Gt, G.mask_to_device(mi), G.mask_to_device(mo)).cpu().numpy()
    ref, _ = oracle_mod.factmask(W.bits_of(A), W.bits_of(Gt), mi, mo, dtype="f32")
    rel = _max_rel(out, ref)
    assert rel <= 4e-6, rel


def test_fim_positive_operands(G, oracle_mod):
    X = _positive((512, 192), 6)
    F = G.grass_fim(X).cpu().numpy()
    ref, _ = oracle_mod.fim(X.cpu().numpy())
    rel = _max_rel(F, ref)
    assert rel <= 4e-6, rel


def test_fim_accuracy_at_n_4096(G, oracle_mod):
    g = torch.Generator(device="cuda")
    g.manual_seed(11)
    X = torch.randn((4096, 256), generator=g, device="cuda")
    F = G.grass_fim(X).cpu().numpy()
    ref, absum = oracle_mod.fim(X.cpu().numpy())
    rel = check_close(F, ref, absum, 1e-4, 4096 + 64, eps=2.0 ** -23, what="fim n=4096")
    assert rel <= 1e-3
    assert_accurate(F, ref, 2e-5, what="fim n=4096")


@pytest.mark.parametrize("nprod,limit", [(4, 4e-6), (3, 4e-6)])
def test_fewer_partial_products_stay_unbiased(G, oracle_mod, tune, nprod, limit):
    """The pieces are rounded to nearest, so what two pieces leave out has either sign (at most 2^-17 of a
    product): with four products (no lo piece at all), and with three (mid*mid dropped as well), sums over
    operands of one sign are still right to about 1e-6.  Six stay the default: they make every single product
    fp32-accurate, these only the sums, and the kernels' time does not depend on the count (the split of the
    operands sets the pace, not the tensor pipe)."""
    tr, te = _positive((300, 512), 1), _positive((70, 512), 2)
    ref, _ = oracle_mod.score(tr.cpu().numpy(), te.cpu().numpy())
    tune(score_splits=1, split_products=nprod)
    rel = _max_rel(G.grass_score(tr, te).cpu().numpy(), ref)
    assert rel <= limit, (nprod, rel)


def test_worst_case_operands_show_what_the_last_two_products_buy(G, tune):
    """x = 1 + 2^-9 + 2^-18 in every entry: the third bf16 piece of each operand is 2^-18 with the same sign
    everywhere, so dropping it (four products) errs by 2 * 2^-18 = 7.6e-6 of every product and of their sum
    (closed form D x^2); all six products leave only the accumulator's truncation."""
    x = 1.0 + 2.0 ** -9 + 2.0 ** -18
    D = 512
    tr = torch.full((256, D), x, device="cuda")
    te = torch.full((64, D), x, device="cuda")
    assert float(tr[0, 0].double().item()) == x                      # exact in fp32
    exact = D * x * x
    tune(score_splits=1)
    rel6 = float((G.grass_score(tr, te).double() - exact).abs().max().item() / exact)
    assert rel6 <= 4e-6, rel6
    tune(split_products=4)
    rel4 = float((G.grass_score(tr, te).double() - exact).abs().max().item() / exact)
    assert 5e-6 <= rel4 <= 2e-5, rel4
