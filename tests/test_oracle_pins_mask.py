"""Pins of the oracle's stand-alone sparsification (Section 3.2) and its factorised form (CPU only)."""
import numpy as np
import torch


def _bf16(rng, shape):
    x = torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)
    return x.view(torch.uint16).numpy().copy(), x.float().numpy().astype(np.float64)


def test_mask_is_the_selection_matrix_product(oracle_mod):
    rng = np.random.default_rng(0)
    n, p, kp = 5, 40, 11
    g = rng.standard_normal((n, p)).astype(np.float32)
    idx = oracle_mod.random_mask(p, kp, 3)
    M = np.zeros((kp, p))
    M[np.arange(kp), idx] = 1.0                  # one non-repeating 1 per row
    np.testing.assert_array_equal(oracle_mod.mask(g, idx), g.astype(np.float64) @ M.T)
    # row stride: columns past p are never read
    wide = np.full((n, p + 3), np.nan, dtype=np.float32)
    wide[:, :p] = g
    np.testing.assert_array_equal(oracle_mod.mask(wide, idx, p=p), g.astype(np.float64)[:, idx])
    # bf16 decode
    gb, gf = _bf16(rng, (n, p))
    np.testing.assert_array_equal(oracle_mod.mask(gb, idx, dtype="bf16"), gf[:, idx])


def test_factmask_is_eq2_with_selection_matrices(oracle_mod):
    rng = np.random.default_rng(1)
    B, T, d_in, d_out, kin, kout = 3, 9, 12, 10, 5, 4
    Ab, Af = _bf16(rng, (B, T, d_in))
    Gb, Gf = _bf16(rng, (B, T, d_out))
    mi = oracle_mod.random_mask(d_in, kin, 1)
    mo = oracle_mod.random_mask(d_out, kout, 2)
    out, ab = oracle_mod.factmask(Ab, Gb, mi, mo)
    # (P_in (x) P_out) vec(sum_t a_t (x) b_t) with P = selection matrices: gather of the full gradient
    full = np.einsum("bti,bto->bio", Af, Gf).reshape(B, d_in * d_out)
    kmask = (mi[:, None].astype(np.int64) * d_out + mo[None, :]).reshape(-1)
    np.testing.assert_allclose(out, full[:, kmask], rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(ab, np.einsum("bti,bto->bio", np.abs(Af), np.abs(Gf)).reshape(B, -1)[:, kmask], rtol=1e-13)
    # per-sample gradient identity (Eq. 1): the block is a sub-matrix of G^T A, transposed (input-major)
    for b in range(B):
        dW = Gf[b].T @ Af[b]                                   # d_out x d_in
        np.testing.assert_allclose(out[b].reshape(kin, kout), dW[np.ix_(mo, mi)].T, rtol=1e-12, atol=1e-14)
    # FactGraSS = SJLT of this block (Section 3.3.2): both halves of the composition are pinned separately
    fg, _ = oracle_mod.factgrass(Ab, Gb, mi, mo, 7, 2, 99)
    hi = out.astype(np.float32)
    lo = (out - hi).astype(np.float32)
    ref = oracle_mod.grass(hi, None, 7, 2, 99)[0] + oracle_mod.grass(lo, None, 7, 2, 99)[0]
    np.testing.assert_allclose(fg, ref, rtol=1e-12, atol=1e-13)
