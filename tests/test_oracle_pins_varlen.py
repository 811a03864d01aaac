"""Pins of the oracle's sequence-length-aware FactGraSS (CPU only).

Eq. 2 sums over the tokens of one sample, so a batch of samples with different lengths is
the plain FactGraSS applied sample by sample to that sample's own tokens.  The function is pinned
to the already pinned oracle_factgrass (full length, zero-gradient padding, per-sample slices)
and, independently of it, to the dense projection matrix applied to numpy's masked A^T G."""
import numpy as np
import torch


def _bf16(rng, shape):
    x = torch.from_numpy(rng.standard_normal(shape).astype(np.float32)).to(torch.bfloat16)
    return x.view(torch.uint16).numpy().copy(), x.float().numpy().astype(np.float64)


def _setup(oracle_mod, seed=3):
    rng = np.random.default_rng(seed)
    B, T, d_in, d_out, kin, kout, k = 4, 11, 14, 18, 6, 5, 13
    Ab, Af = _bf16(rng, (B, T, d_in))
    Gb, Gf = _bf16(rng, (B, T, d_out))
    mi = oracle_mod.random_mask(d_in, kin, 1)
    mo = oracle_mod.random_mask(d_out, kout, 2)
    return B, T, d_in, d_out, kin, kout, k, Ab, Af, Gb, Gf, mi, mo


def test_full_length_equals_plain_factgrass(oracle_mod):
    B, T, d_in, d_out, kin, kout, k, Ab, Af, Gb, Gf, mi, mo = _setup(oracle_mod)
    for s in (1, 3):
        ref, rab = oracle_mod.factgrass(Ab, Gb, mi, mo, k, s, 99)
        out, ab = oracle_mod.factgrass_varlen(Ab.reshape(B * T, d_in), Gb.reshape(B * T, d_out), mi, mo, k, s, 99,
                                              np.arange(B) * T, np.full(B, T))
        np.testing.assert_allclose(out, ref, rtol=1e-13, atol=1e-15)
        np.testing.assert_allclose(ab, rab, rtol=1e-13)


def test_short_samples_equal_zero_gradient_padding(oracle_mod):
    """Tokens past a sample's length are ignored: the same as padding tokens whose output gradient is 0."""
    B, T, d_in, d_out, kin, kout, k, Ab, Af, Gb, Gf, mi, mo = _setup(oracle_mod, 4)
    lens = np.array([T, 0, 5, 1])
    Gz = Gb.copy()
    for b in range(B):
        Gz[b, lens[b]:] = 0
    ref, rab = oracle_mod.factgrass(Ab, Gz, mi, mo, k, 1, 5)
    out, ab = oracle_mod.factgrass_varlen(Ab.reshape(B * T, d_in), Gb.reshape(B * T, d_out), mi, mo, k, 1, 5,
                                          np.arange(B) * T, lens)
    np.testing.assert_allclose(out, ref, rtol=1e-13, atol=1e-15)
    np.testing.assert_allclose(ab, rab, rtol=1e-13, atol=1e-15)
    assert np.all(out[1] == 0) and np.all(ab[1] == 0)            # an empty sample compresses to zero


def test_packed_batch_equals_per_sample_calls(oracle_mod):
    B, T, d_in, d_out, kin, kout, k, Ab, Af, Gb, Gf, mi, mo = _setup(oracle_mod, 5)
    lens = np.array([3, 11, 7, 2])
    begin = np.concatenate([[0], np.cumsum(lens)[:-1]])
    Ap = np.concatenate([Ab[b, :lens[b]] for b in range(B)])
    Gp = np.concatenate([Gb[b, :lens[b]] for b in range(B)])
    out, ab = oracle_mod.factgrass_varlen(np.ascontiguousarray(Ap), np.ascontiguousarray(Gp), mi, mo, k, 2, 8, begin, lens)
    for b in range(B):
        ref, rab = oracle_mod.factgrass(np.ascontiguousarray(Ab[b:b + 1, :lens[b]]),
                                        np.ascontiguousarray(Gb[b:b + 1, :lens[b]]), mi, mo, k, 2, 8)
        np.testing.assert_allclose(out[b], ref[0], rtol=1e-13, atol=1e-15)
        np.testing.assert_allclose(ab[b], rab[0], rtol=1e-13, atol=1e-15)
    # samples may be listed in any order and may leave gaps between them
    order = np.array([2, 0, 3, 1])
    o2, _ = oracle_mod.factgrass_varlen(np.ascontiguousarray(Ap), np.ascontiguousarray(Gp), mi, mo, k, 2, 8,
                                        begin[order], lens[order])
    np.testing.assert_allclose(o2, out[order], rtol=0, atol=0)


def test_against_dense_projection_of_numpy_contraction(oracle_mod):
    """Independent of oracle_factgrass: out_b = P vec(A_b[:, mask_in]^T G_b[:, mask_out]) with the
    explicit k x (kin*kout) matrix P built from the (bucket, sign) table."""
    B, T, d_in, d_out, kin, kout, k, Ab, Af, Gb, Gf, mi, mo = _setup(oracle_mod, 6)
    s, seed = 2, 31
    lens = np.array([T, 4, 9, 6])
    bucket, sign = oracle_mod.sjlt_table(k, s, seed, kin * kout)
    P = np.zeros((k, kin * kout))
    for j in range(kin * kout):
        for r in range(s):
            P[bucket[j * s + r], j] += sign[j * s + r] / np.sqrt(s)
    out, ab = oracle_mod.factgrass_varlen(Ab.reshape(B * T, d_in), Gb.reshape(B * T, d_out), mi, mo, k, s, seed,
                                          np.arange(B) * T, lens)
    for b in range(B):
        blk = Af[b, :lens[b]][:, mi].T @ Gf[b, :lens[b]][:, mo]          # kin x kout, input-major flattening
        np.testing.assert_allclose(out[b], P @ blk.reshape(-1), rtol=1e-12, atol=1e-13)
        ablk = np.abs(Af[b, :lens[b]][:, mi]).T @ np.abs(Gf[b, :lens[b]][:, mo])
        np.testing.assert_allclose(ab[b], np.abs(P) @ ablk.reshape(-1), rtol=1e-12, atol=1e-13)
