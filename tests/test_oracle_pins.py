"""CPU pins for the oracle: each test ties one part of ``oracle/`` to something
the paper or the mathematics fixes, not to the oracle's own formula."""
import math

import numpy as np
import pytest
import torch

M64 = (1 << 64) - 1


# ------------------------------------------------------------------ hash family

def test_hash_counter_layout(oracle_mod):
    """Draw r of position j uses counter j*s + r + 1: the s draws of all positions
    tile the SplitMix64 stream without gaps or overlaps."""
    seed, s = 99, 3
    stream = [oracle_mod.sjlt_hash(seed, 1, n, 0) for n in range(12)]
    got = [oracle_mod.sjlt_hash(seed, s, j, r) for j in range(4) for r in range(s)]
    assert got == stream


def test_table_matches_hash_and_range(oracle_mod):
    k, s, seed, kp = 37, 2, 5, 500
    bucket, sign = oracle_mod.sjlt_table(k, s, seed, kp)
    assert bucket.max() < k and set(np.unique(sign)) <= {-1, 1}
    for j in (0, 1, 17, 499):
        for r in range(s):
            h = oracle_mod.sjlt_hash(seed, s, j, r)
            assert bucket[j * s + r] == ((h >> 32) * k) >> 32      # multiply-shift range reduction
            assert sign[j * s + r] == (-1 if h & 1 else 1)


def test_bucket_uniformity_sign_balance_collisions(oracle_mod):
    k, kp = 256, 1 << 16
    bucket, sign = oracle_mod.sjlt_table(k, 1, 0xABCDEF, kp)
    counts = np.bincount(bucket, minlength=k)
    chi2 = ((counts - kp / k) ** 2 / (kp / k)).sum()
    # chi-square with 255 dof: mean 255, sd ~22.6; 5 sd band
    assert abs(chi2 - (k - 1)) < 5 * math.sqrt(2 * (k - 1))
    assert abs(int(sign.astype(np.int64).sum())) < 5 * math.sqrt(kp)
    # pairwise collision rate ~ 1/k
    a, b = bucket[: kp // 2], bucket[kp // 2:]
    rate = (a == b).mean()
    assert abs(rate - 1 / k) < 5 * math.sqrt((1 / k) / (kp // 2))
    # bucket and sign independent
    assert abs(np.corrcoef(bucket.astype(float), sign.astype(float))[0, 1]) < 0.02


# ------------------------------------------------------------------ SJLT

def _dense_P(oracle_mod, k, s, seed, kp):
    """Materialise the sparse projection matrix: column j holds s entries +-1/sqrt(s)."""
    bucket, sign = oracle_mod.sjlt_table(k, s, seed, kp)
    P = np.zeros((k, kp))
    Pabs = np.zeros((k, kp))       # same entries without signs (draws that collide do not cancel)
    for j in range(kp):
        for r in range(s):
            P[bucket[j * s + r], j] += sign[j * s + r] / math.sqrt(s)
            Pabs[bucket[j * s + r], j] += 1 / math.sqrt(s)
    return P, Pabs


@pytest.mark.parametrize("s", [1, 2, 4])
def test_sjlt_equals_materialised_matrix(oracle_mod, s):
    rng = np.random.default_rng(1)
    n, p, k, seed = 5, 97, 13, 42 + s
    g = rng.integers(-8, 9, size=(n, p)).astype(np.float32)     # small integers: sums exact
    out, absum = oracle_mod.grass(g, None, k, s, seed)
    P, Pabs = _dense_P(oracle_mod, k, s, seed, p)
    np.testing.assert_allclose(out, g.astype(np.float64) @ P.T, rtol=0, atol=1e-12)
    np.testing.assert_allclose(absum, np.abs(g).astype(np.float64) @ Pabs.T, rtol=0, atol=1e-12)
    # every column: s non-zeros of magnitude 1/sqrt(s), counted with multiplicity
    np.testing.assert_allclose(Pabs.sum(axis=0), s / math.sqrt(s), atol=1e-12)


def test_one_hot_reads_out_the_table(oracle_mod):
    p, k, seed = 64, 11, 7
    bucket, sign = oracle_mod.sjlt_table(k, 1, seed, p)
    out, _ = oracle_mod.grass(np.eye(p, dtype=np.float32), None, k, 1, seed)
    for j in range(p):
        expect = np.zeros(k)
        expect[bucket[j]] = sign[j]
        assert np.array_equal(out[j], expect)


def test_linearity(oracle_mod):
    rng = np.random.default_rng(2)
    x = rng.integers(-100, 100, (1, 300)).astype(np.float32)
    y = rng.integers(-100, 100, (1, 300)).astype(np.float32)
    f = lambda v: oracle_mod.grass(np.ascontiguousarray(v, dtype=np.float32), None, 17, 2, 3)[0]
    np.testing.assert_allclose(f(3 * x - 2 * y), 3 * f(x) - 2 * f(y), rtol=0, atol=1e-9)


@pytest.mark.parametrize("s", [1, 2, 4])
def test_jl_moments_over_seeds(oracle_mod, s):
    """E||Sx||^2 = ||x||^2 (this is what fixes the 1/sqrt(s) scale) and, for s = 1 with a
    fully random hash, Var||Sx||^2 = (2/k)(||x||_2^4 - ||x||_4^4); E<Sx,Sy> = <x,y>."""
    rng = np.random.default_rng(3)
    p, k, nseeds = 200, 32, 2000
    x = rng.standard_normal((1, p)).astype(np.float32)
    y = (0.5 * x + rng.standard_normal((1, p))).astype(np.float32)
    xy = np.concatenate([x, y])
    n2, ip = [], []
    for seed in range(nseeds):
        o, _ = oracle_mod.grass(xy, None, k, s, 1000 + seed, want_absum=False)
        n2.append((o[0] ** 2).sum())
        ip.append((o[0] * o[1]).sum())
    n2, ip = np.array(n2), np.array(ip)
    x64 = x.astype(np.float64)[0]
    true_n2 = (x64 ** 2).sum()
    assert abs(n2.mean() - true_n2) < 4 * n2.std() / math.sqrt(nseeds)
    true_ip = float(x64 @ y.astype(np.float64)[0])
    assert abs(ip.mean() - true_ip) < 4 * ip.std() / math.sqrt(nseeds)
    if s == 1:
        var = (2 / k) * (true_n2 ** 2 - (x64 ** 4).sum())
        assert abs(n2.var() / var - 1) < 0.15


# ------------------------------------------------------------------ mask

def test_random_mask_is_a_selection_matrix(oracle_mod):
    p, kp = 1000, 137
    idx = oracle_mod.random_mask(p, kp, 11)
    assert idx.dtype == np.uint32 and idx.size == kp
    assert np.all(np.diff(idx.astype(np.int64)) > 0) and idx.max() < p   # distinct, ascending
    # gather == M g with the explicit binary M (one 1 per row)
    M = np.zeros((kp, p))
    M[np.arange(kp), idx] = 1
    g = np.random.default_rng(4).standard_normal((3, p)).astype(np.float32)
    k, seed = 1 << 12, 0
    # k >> k' and s=1: compare through an identity-mask call on M g
    out_mask, _ = oracle_mod.grass(g, idx, k, 1, seed)
    out_Mg, _ = oracle_mod.grass(np.ascontiguousarray((g @ M.T).astype(np.float32)), None, k, 1, seed)
    assert np.array_equal(out_mask, out_Mg)


def test_random_mask_edge_cases(oracle_mod):
    assert np.array_equal(oracle_mod.random_mask(50, 50, 9), np.arange(50, dtype=np.uint32))
    assert oracle_mod.random_mask(50, 0, 9).size == 0
    with pytest.raises(ValueError):
        oracle_mod.random_mask(10, 11, 0)
    assert not np.array_equal(oracle_mod.random_mask(10_000, 100, 1), oracle_mod.random_mask(10_000, 100, 2))


def test_random_mask_uniform_inclusion(oracle_mod):
    p, kp, trials = 60, 12, 6000
    counts = np.zeros(p)
    pair = 0
    for seed in range(trials):
        idx = oracle_mod.random_mask(p, kp, seed)
        counts[idx] += 1
        pair += (0 in idx) and (p - 1 in idx)
    # each coordinate is included w.p. k'/p
    sd = math.sqrt(trials * (kp / p) * (1 - kp / p))
    assert np.all(np.abs(counts - trials * kp / p) < 4.5 * sd)
    # a pair w.p. k'(k'-1)/(p(p-1)): rules out sampling with replacement + dedup
    pp = kp * (kp - 1) / (p * (p - 1))
    assert abs(pair - trials * pp) < 4.5 * math.sqrt(trials * pp * (1 - pp))


def test_grass_identity_mask_is_plain_sjlt(oracle_mod):
    """k' = p reduces GraSS to SJLT (Section 3.3.1)."""
    g = np.random.default_rng(5).standard_normal((4, 200)).astype(np.float32)
    a, _ = oracle_mod.grass(g, np.arange(200, dtype=np.uint32), 16, 1, 8)
    b, _ = oracle_mod.grass(g, None, 16, 1, 8)
    assert np.array_equal(a, b)


def test_row_stride_and_bf16_decode(oracle_mod):
    rng = np.random.default_rng(6)
    p, ld = 90, 128
    g = np.full((3, ld), np.nan, dtype=np.float32)
    g[:, :p] = rng.standard_normal((3, p))
    a, _ = oracle_mod.grass(g, None, 8, 1, 1, p=p)
    b, _ = oracle_mod.grass(np.ascontiguousarray(g[:, :p]), None, 8, 1, 1)
    assert np.array_equal(a, b)
    # bf16 bit patterns decode as torch decodes them
    t = torch.randn(3, p).to(torch.bfloat16)
    bits = t.view(torch.uint16).numpy()
    c, _ = oracle_mod.grass(bits, None, 8, 1, 1, dtype="bf16")
    d, _ = oracle_mod.grass(t.float().numpy(), None, 8, 1, 1)
    assert np.array_equal(c, d)


# ------------------------------------------------------------------ Eq. 1 / FactGraSS

def test_per_sample_gradient_identity_finite_differences():
    """Eq. 1: vec(DW) = sum_t a_t (x) b_t, i.e. DW = G^T A (d_out x d_in), checked against
    central differences of l(W) = sum_t <c_t, W a_t> whose pre-activation gradient is c_t."""
    rng = np.random.default_rng(7)
    T, d_in, d_out = 6, 5, 7
    A = rng.standard_normal((T, d_in))
    C = rng.standard_normal((T, d_out))
    W = rng.standard_normal((d_out, d_in))
    loss = lambda W_: sum(C[t] @ (W_ @ A[t]) for t in range(T))
    fd = np.zeros_like(W)
    eps = 1e-5
    for i in range(d_out):
        for j in range(d_in):
            E = np.zeros_like(W)
            E[i, j] = eps
            fd[i, j] = (loss(W + E) - loss(W - E)) / (2 * eps)
    kron = sum(np.kron(A[t], C[t]) for t in range(T))            # input-major flattening
    # column-stacking vec of the d_out x d_in matrix: entry (o, i) at i*d_out + o
    np.testing.assert_allclose(kron.reshape(d_in, d_out).T, fd, rtol=1e-6, atol=1e-8)
    np.testing.assert_allclose(kron.reshape(d_in, d_out).T, C.T @ A, rtol=1e-12, atol=1e-12)


def _bf16(rng, shape, scale=1.0):
    t = (torch.from_numpy(rng.standard_normal(shape).astype(np.float32)) * scale).to(torch.bfloat16)
    return t.view(torch.uint16).numpy().copy(), t.float().numpy().astype(np.float64)


def test_factgrass_equals_grass_with_kronecker_mask(oracle_mod):
    """Eq. 2 with selection matrices: FactGraSS must equal GraSS applied to the fully
    materialised flattened gradient sum_t a_t (x) b_t under the mask
    idx[a*kout + c] = mask_in[a]*d_out + mask_out[c]."""
    rng = np.random.default_rng(8)
    B, T, d_in, d_out, kin, kout, k = 3, 9, 12, 10, 5, 4, 7
    Ab, Af = _bf16(rng, (B, T, d_in))
    Gb, Gf = _bf16(rng, (B, T, d_out))
    mi = oracle_mod.random_mask(d_in, kin, 1)
    mo = oracle_mod.random_mask(d_out, kout, 2)
    for s in (1, 2):
        out, absum = oracle_mod.factgrass(Ab, Gb, mi, mo, k, s, 77)
        full = np.einsum("bti,bto->bio", Af, Gf).reshape(B, d_in * d_out)   # exact in float64
        kmask = (mi[:, None].astype(np.int64) * d_out + mo[None, :]).reshape(-1).astype(np.uint32)
        assert np.all(np.diff(kmask.astype(np.int64)) > 0)
        # float32 cannot hold the exact sums: run GraSS on hi + lo float32 parts and add (linearity)
        hi = full.astype(np.float32)
        lo = (full - hi).astype(np.float32)
        ref = oracle_mod.grass(hi, kmask, k, s, 77)[0] + oracle_mod.grass(lo, kmask, k, s, 77)[0]
        np.testing.assert_allclose(out, ref, rtol=1e-12, atol=1e-13)
        absfull = np.einsum("bti,bto->bio", np.abs(Af), np.abs(Gf)).reshape(B, -1)
        ahi = absfull.astype(np.float32)
        aref = oracle_mod.grass(ahi, kmask, k, s, 77)[1] + oracle_mod.grass((absfull - ahi).astype(np.float32), kmask, k, s, 77)[1]
        np.testing.assert_allclose(absum, aref, rtol=1e-6)


def test_factgrass_invariants(oracle_mod):
    rng = np.random.default_rng(9)
    B, T, d_in, d_out, kin, kout, k, seed = 2, 8, 16, 24, 6, 5, 9, 5
    Ab, Af = _bf16(rng, (B, T, d_in))
    Gb, Gf = _bf16(rng, (B, T, d_out))
    mi = oracle_mod.random_mask(d_in, kin, 3)
    mo = oracle_mod.random_mask(d_out, kout, 4)
    base, _ = oracle_mod.factgrass(Ab, Gb, mi, mo, k, 1, seed)
    # T = 1: SJLT(a' (x) b')
    o1, _ = oracle_mod.factgrass(np.ascontiguousarray(Ab[:, :1]), np.ascontiguousarray(Gb[:, :1]), mi, mo, k, 1, seed)
    kr = np.stack([np.kron(Af[b, 0, mi], Gf[b, 0, mo]) for b in range(B)])
    hi = kr.astype(np.float32)
    ref = oracle_mod.grass(hi, None, k, 1, seed)[0] + oracle_mod.grass((kr - hi).astype(np.float32), None, k, 1, seed)[0]
    np.testing.assert_allclose(o1, ref, rtol=1e-12, atol=1e-14)
    # appended tokens with zero output-gradient change nothing (padding)
    Apad = np.concatenate([Ab, Ab[:, :3]], axis=1)
    Gpad = np.concatenate([Gb, np.zeros_like(Gb[:, :3])], axis=1)
    o2, _ = oracle_mod.factgrass(np.ascontiguousarray(Apad), np.ascontiguousarray(Gpad), mi, mo, k, 1, seed)
    assert np.array_equal(o2, base)
    # token order does not matter (up to rounding order)
    perm = rng.permutation(T)
    o3, _ = oracle_mod.factgrass(np.ascontiguousarray(Ab[:, perm]), np.ascontiguousarray(Gb[:, perm]), mi, mo, k, 1, seed)
    np.testing.assert_allclose(o3, base, rtol=1e-12, atol=1e-14)
    # splitting the token sum and adding the compressed halves (linearity of SJLT)
    h1, _ = oracle_mod.factgrass(np.ascontiguousarray(Ab[:, :5]), np.ascontiguousarray(Gb[:, :5]), mi, mo, k, 1, seed)
    h2, _ = oracle_mod.factgrass(np.ascontiguousarray(Ab[:, 5:]), np.ascontiguousarray(Gb[:, 5:]), mi, mo, k, 1, seed)
    np.testing.assert_allclose(h1 + h2, base, rtol=1e-12, atol=1e-14)
    # swapping the factor roles changes the flattening: a transposed operand must be caught
    o4, _ = oracle_mod.factgrass(Ab, Gb, mi[::-1].copy(), mo, k, 1, seed)
    assert not np.allclose(o4, base)


# ------------------------------------------------------------------ score

def test_score_is_the_inner_product(oracle_mod):
    rng = np.random.default_rng(10)
    tr = rng.standard_normal((7, 33)).astype(np.float32)
    te = rng.standard_normal((4, 33)).astype(np.float32)
    sc, ab = oracle_mod.score(tr, te)
    np.testing.assert_allclose(sc, tr.astype(np.float64) @ te.astype(np.float64).T, rtol=1e-13, atol=1e-13)
    np.testing.assert_allclose(ab, np.abs(tr).astype(np.float64) @ np.abs(te).astype(np.float64).T, rtol=1e-13)
    assert sc.shape == (7, 4)                                     # train-major


def test_score_kronecker_identity(oracle_mod):
    """<a (x) b, a' (x) b'> = <a, a'> <b, b'> (appendix, factorised Selective Mask)."""
    rng = np.random.default_rng(11)
    a, a2 = rng.integers(-4, 5, (2, 6)).astype(np.float32)
    b, b2 = rng.integers(-4, 5, (2, 5)).astype(np.float32)
    sc, _ = oracle_mod.score(np.kron(a, b)[None].astype(np.float32), np.kron(a2, b2)[None].astype(np.float32))
    assert sc[0, 0] == float(a @ a2) * float(b @ b2)


# ------------------------------------------------------------------ planted mistakes

def test_pins_catch_a_dropped_sign(oracle_mod):
    """The materialised-matrix pin is sensitive: with all signs forced to +1 the
    comparison made in test_sjlt_equals_materialised_matrix would not hold."""
    rng = np.random.default_rng(12)
    g = rng.integers(1, 9, size=(1, 50)).astype(np.float32)
    out, absum = oracle_mod.grass(g, None, 5, 1, 3)
    assert not np.array_equal(out, absum)          # signs do flip some terms
    assert np.all(np.abs(out) <= absum + 1e-12)
