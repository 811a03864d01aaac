"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle, element by
element, on the same seeded inputs.  Indices, buckets and signs bit-exact; values within
the tolerance rule of tests/parity.py."""
import dataclasses

import numpy as np
import pytest
import torch

from parity import check_close, max_bin_load

pytestmark = pytest.mark.gpu

TOL_F32, TOL_BF16 = 1e-4, 2e-2
EPS_TC = 2.0 ** -23


@pytest.fixture(scope="module")
def G():
    import paper_2505_18976_b200 as g
    g.lib()
    return g


@pytest.fixture(scope="module")
def W():
    from paper_2505_18976_b200 import workloads
    return workloads


def _dev_mask(G, idx):
    return G.mask_to_device(idx)


# ------------------------------------------------------------------ hash, bit-exact

@pytest.mark.parametrize("k,s,seed,kp", [(2048, 1, 0x5EED + 1, 8192), (4096, 1, 0x5EED + 2, 65536),
                                         (1000003, 3, 7, 5000), (1, 2, 9, 100), (4294967295, 1, 2 ** 64 - 1, 4096)])
def test_device_hash_table_bit_exact(G, oracle_mod, k, s, seed, kp):
    b, sg = G.grass_sjlt_table(k, s, seed, kp)
    ob, osg = oracle_mod.sjlt_table(k, s, seed, kp)
    assert np.array_equal(b.cpu().numpy().view(np.uint32), ob)
    assert np.array_equal(sg.cpu().numpy(), osg)


def test_one_hot_through_grass_compress_reads_the_table(G, oracle_mod):
    """e_j in -> sign(j) e_{bucket(j)} out, through the compress kernel itself."""
    p, k, seed = 1536, 257, 0xBEEF
    out = G.grass_compress(torch.eye(p, device="cuda"), None, k, 1, seed).cpu().numpy()
    ob, osg = oracle_mod.sjlt_table(k, 1, seed, p)
    expect = np.zeros((p, k), dtype=np.float32)
    expect[np.arange(p), ob] = osg
    assert np.array_equal(out, expect)


def test_one_hot_through_factgrass_reads_the_table(G, oracle_mod, fg_path):
    """T = 1, A = e_a, G = e_c: the only non-zero block entry sits at q = a*kout + c."""
    kin, kout, k, seed = 24, 40, 97, 11
    d_in, d_out = 64, 96
    mi = oracle_mod.random_mask(d_in, kin, 1)
    mo = oracle_mod.random_mask(d_out, kout, 2)
    pairs = [(0, 0), (3, 7), (23, 39), (10, 0), (0, 39)]
    A = torch.zeros(len(pairs), 1, d_in, dtype=torch.bfloat16, device="cuda")
    Gt = torch.zeros(len(pairs), 1, d_out, dtype=torch.bfloat16, device="cuda")
    for n, (a, c) in enumerate(pairs):
        A[n, 0, int(mi[a])] = 1.0
        Gt[n, 0, int(mo[c])] = 1.0
    out = G.factgrass_compress(A, Gt, _dev_mask(G, mi), _dev_mask(G, mo), k, 1, seed).cpu().numpy()
    ob, osg = oracle_mod.sjlt_table(k, 1, seed, kin * kout)
    for n, (a, c) in enumerate(pairs):
        e = np.zeros(k, dtype=np.float32)
        e[ob[a * kout + c]] = osg[a * kout + c]
        assert np.array_equal(out[n], e), (a, c)


# ------------------------------------------------------------------ grass_compress

def _grass_case(G, W, oracle_mod, n, p, kprime, k, s=1, dtype=torch.float32, ld=None, identity=False,
                zero_prob=0.8, dist="normal", scale=1.0, seed=0, data_seed=5):
    g = W.dense_gradients(n, p, zero_prob, dist, scale, data_seed, device="cuda", dtype=dtype, ld=ld)
    idx = None if identity else oracle_mod.random_mask(p, kprime, seed)
    didx = None if identity else _dev_mask(G, idx)
    host = W.bits_of(g)
    ref, absum = oracle_mod.grass(host, idx, k, s, seed + 99, dtype="f32" if dtype == torch.float32 else "bf16", p=p)
    kp = p if identity else kprime
    ob, _ = oracle_mod.sjlt_table(k, s, seed + 99, kp)
    chain = max_bin_load(ob, k) + 16
    rel = 0.0
    # both kernels: element gathers, and whole row segments staged in shared memory wherever the operands allow
    # (a mask, 16-byte aligned rows, at most 8 segments per row); the launch-shape overrides of a test stay in force
    for rows in ((0,) if identity else (0, 1)):
        with G.tuning(compress_rows=rows):
            status = torch.zeros(1, dtype=torch.int32, device="cuda")
            out = torch.full((n, k), 7.0, device="cuda")
            G.grass_compress(g, didx, k, s, seed + 99, out=out, p=p, dev_status=status)
            torch.cuda.synchronize()
            assert int(status.item()) == 0
        rel = max(rel, check_close(out.cpu().numpy(), ref, absum, TOL_F32, chain,
                                   what=f"grass rows={rows} n={n} p={p} k'={kp} k={k} s={s}"))
    return rel


@pytest.mark.parametrize("n,p,kprime,k", [
    (64, 65_536, 8_192, 2_048),        # config 1 scaled in n
    (16, 1 << 20, 16_384, 4_096),      # config 2 scaled in p and k'
    (7, 10_007, 1_237, 333),           # nothing a multiple of anything
    (3, 4_096, 4_096, 64),             # mask covers every coordinate
    (5, 70_000, 33, 4_096),            # fewer masked coordinates than a warp
    (9, 300_000, 50_000, 60_000),      # k too large for shared-memory bins: global path
    (1, 50_000, 9_999, 1),             # single output bin
])
def test_grass_compress_parity(G, W, oracle_mod, n, p, kprime, k):
    _grass_case(G, W, oracle_mod, n, p, kprime, k)


@pytest.mark.parametrize("s", [2, 4])
def test_grass_compress_s_gt_1(G, W, oracle_mod, s):
    _grass_case(G, W, oracle_mod, 6, 20_000, 5_000, 512, s=s)


def test_grass_compress_identity_mask_and_stride(G, W, oracle_mod):
    _grass_case(G, W, oracle_mod, 10, 65_536, 65_536, 2_048, identity=True)
    _grass_case(G, W, oracle_mod, 5, 9_001, 700, 100, ld=9_016)                  # ld > p, tail is NaN
    _grass_case(G, W, oracle_mod, 5, 9_001, 9_001, 100, ld=9_016, identity=True)


@pytest.mark.parametrize("zero_prob", [0.0, 0.5, 0.9, 0.99, 0.999])
def test_plain_sjlt_over_input_sparsity(G, W, oracle_mod, tune, zero_prob):
    """Identity mask on vector-aligned rows: rounds of loads with few non-zeros go through the per-warp queue, fuller
    ones are hashed in place; one and two samples per CTA, s = 1 and 2, fp32 and bf16, a ragged tail, an odd k,
    and a k whose bins do not fit in shared memory."""
    for S in (1, 2):
        tune(compress_samples=S)
        _grass_case(G, W, oracle_mod, 9, 131_072, 131_072, 4_096, identity=True, zero_prob=zero_prob)
        _grass_case(G, W, oracle_mod, 5, 40_004, 40_004, 777, s=2, identity=True, zero_prob=zero_prob)
        _grass_case(G, W, oracle_mod, 4, 33_000, 33_000, 512, identity=True, zero_prob=zero_prob, dtype=torch.bfloat16)
    tune(compress_samples=None)
    _grass_case(G, W, oracle_mod, 3, 70_000, 70_000, 60_000, identity=True, zero_prob=zero_prob)
    tune(compress_jsplit=5)
    _grass_case(G, W, oracle_mod, 3, 50_000, 50_000, 300, identity=True, zero_prob=zero_prob)


def test_grass_compress_seeded_shape_sweep(G, W, oracle_mod):
    """Seeded random shapes: row lengths, strides with a NaN tail beyond p, mask sizes from a handful to every
    coordinate, output lengths from one bin to more bins than masked coordinates, one to three draws, both dtypes,
    sparse and dense rows."""
    rng = np.random.default_rng(4321)
    for case in range(12):
        p = int(rng.integers(40, 120_000))
        kprime = int(rng.choice([1, 31, 33, p // 7 + 1, p // 2 + 1, p]))
        identity = kprime == p and case % 2 == 0
        _grass_case(G, W, oracle_mod, int(rng.integers(1, 20)), p, kprime, int(rng.integers(1, 6_000)),
                    s=int(rng.choice([1, 1, 2, 3])), dtype=torch.bfloat16 if case % 4 == 1 else torch.float32,
                    ld=p + 8 * int(rng.integers(0, 3)), identity=identity, zero_prob=float(rng.choice([0.0, 0.7, 0.97])),
                    seed=case, data_seed=50 + case)


def test_grass_compress_bf16_input(G, W, oracle_mod):
    _grass_case(G, W, oracle_mod, 12, 100_000, 10_000, 1_024, dtype=torch.bfloat16)


def test_grass_compress_student_t(G, W, oracle_mod):
    _grass_case(G, W, oracle_mod, 8, 1 << 18, 1 << 14, 4_096, zero_prob=0.7, dist="student_t3", scale=1e-2)


@pytest.mark.parametrize("S,js,cluster", [(1, 1, 1), (2, 3, 0), (4, 7, 0), (8, 2, 1), (1, 2, 1), (1, 4, 1), (1, 8, 1),
                                          (2, 4, 1), (1, 8, 0), (1, 20, 1)])
def test_grass_compress_launch_shapes(G, W, oracle_mod, tune, S, js, cluster):
    """Every plan (samples per CTA, position split, cluster or global-atomic reduction) gives the same answer."""
    tune(compress_samples=S, compress_jsplit=js, compress_cluster=cluster)
    _grass_case(G, W, oracle_mod, 11, 40_000, 9_000, 1_000)
    _grass_case(G, W, oracle_mod, 5, 40_000, 9_000, 1_003, s=2)


@pytest.mark.parametrize("threads,loads", [(512, 8), (1024, 8), (256, 16), (1024, 16)])
def test_grass_compress_block_sizes(G, W, oracle_mod, tune, threads, loads):
    """Thread blocks of 512 and 1,024 threads and 16 loads per thread: one round or several, ragged tails, s = 2."""
    tune(compress_threads=threads, compress_loads=loads)
    _grass_case(G, W, oracle_mod, 7, 40_000, 9_000, 1_000)
    _grass_case(G, W, oracle_mod, 3, 70_000, 33_333, 257, s=2)
    _grass_case(G, W, oracle_mod, 200, 20_000, 5_000, 300, dtype=torch.bfloat16)   # a row per SM: whole-row blocks


def test_grass_compress_special_values(G, oracle_mod):
    """All-zero rows give exact zeros; NaN / Inf reach exactly the bins they hash to."""
    n, p, k, seed = 4, 5_000, 64, 3
    g = torch.zeros(n, p, device="cuda")
    g[1, 17] = float("nan")
    g[2, 4_000] = float("inf")
    g[3, :] = 1.0
    out = G.grass_compress(g, None, k, 1, seed).cpu().numpy()
    ob, osg = oracle_mod.sjlt_table(k, 1, seed, p)
    assert np.all(out[0] == 0)
    assert np.isnan(out[1, ob[17]]) and np.all(np.delete(out[1], ob[17]) == 0)
    assert np.isinf(out[2, ob[4_000]]) and out[2, ob[4_000]] == osg[4_000] * np.inf
    assert np.array_equal(out[3], np.bincount(ob, weights=osg.astype(np.float64), minlength=k).astype(np.float32))


def test_grass_compress_empty_and_errors(G, oracle_mod):
    out = G.grass_compress(torch.empty(0, 100, device="cuda"), None, 8, 1, 0)
    assert out.shape == (0, 8)
    # k' = 0: output zeroed
    idx = torch.empty(0, dtype=torch.int32, device="cuda")
    o = torch.full((3, 8), 7.0, device="cuda")
    G.grass_compress(torch.ones(3, 100, device="cuda"), idx, 8, 1, 0, out=o)
    assert torch.all(o == 0)
    # an index >= p (planted on the host) is skipped and flagged, never dereferenced
    p, k = 1_000, 16
    idxh = oracle_mod.random_mask(p, 50, 1)
    bad = idxh.copy()
    bad[-1] = 2_000_000_000
    g = torch.randn(2, p, device="cuda")
    ref_in = g.cpu().numpy().copy()
    ref_in[:, idxh[-1]] = 0        # same as dropping the last masked position
    ref, absum = oracle_mod.grass(ref_in, idxh, k, 1, 5)
    for rows in (0, 1):            # the gather kernel and the row-staging kernel
        with G.tuning(compress_rows=rows):
            st = torch.zeros(1, dtype=torch.int32, device="cuda")
            got = G.grass_compress(g, G.mask_to_device(bad), k, 1, 5, dev_status=st).cpu().numpy()
            assert int(st.item()) & 1
            check_close(got, ref, absum, TOL_F32, 32, what=f"bad index skipped, rows={rows}")
    assert not G.grass_validate_mask(G.mask_to_device(bad), p)
    assert G.grass_validate_mask(G.mask_to_device(idxh), p)
    dup = idxh.copy()
    dup[10] = dup[9]
    assert not G.grass_validate_mask(G.mask_to_device(dup), p)
    with pytest.raises(G.GrassError):
        G.grass_compress(g, G.mask_to_device(idxh), 0, 1, 5)


def test_grass_compress_run_to_run(G, W, oracle_mod):
    """Float atomics reorder sums: repeated runs agree to a few ulps of the bin's mass."""
    g = W.dense_gradients(32, 100_000, 0.5, "normal", 1.0, 3, device="cuda")
    idx = _dev_mask(G, oracle_mod.random_mask(100_000, 20_000, 0))
    a = G.grass_compress(g, idx, 512, 1, 1).cpu().numpy().astype(np.float64)
    for _ in range(3):
        b = G.grass_compress(g, idx, 512, 1, 1).cpu().numpy().astype(np.float64)
        assert np.max(np.abs(a - b)) <= 64 * 2.0 ** -24 * np.abs(a).max() * 8


# ------------------------------------------------------------------ factgrass_compress

def _fact_cfg(W, **kw):
    base = dict(name="t", layers=(W.LinearLayer("l", 96, 160),), B=3, T=70, kin=24, kout=40, k=97, s=1,
                g_dist="normal", g_scale=1e-3, pad_frac=0.0, data_seed=21, mask_seed=4, hash_seed=77)
    base.update(kw)
    return W.FactGrassWorkload(**base)


def _fact_case(G, W, oracle_mod, cfg, l=0, grouped=False, dtype=torch.bfloat16):
    lay = cfg.layers[l]
    A, Gt = W.layer_io(cfg, l, device="cuda", dtype=dtype)
    s_in, s_out = W.layer_mask_seeds(cfg, l)
    mi = oracle_mod.random_mask(lay.d_in, cfg.kin, s_in)
    mo = oracle_mod.random_mask(lay.d_out, cfg.kout, s_out)
    seed = W.layer_hash_seed(cfg, l)
    f32 = dtype == torch.float32
    ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, cfg.k, cfg.s, seed,
                                      dtype="f32" if f32 else "bf16")
    ob, _ = oracle_mod.sjlt_table(cfg.k, cfg.s, seed, cfg.kin * cfg.kout)
    chain = cfg.T + max_bin_load(ob, cfg.k) + 64
    rel = 0.0
    # both kernels: the streaming one, and the cluster one wherever the layer fits it (bf16, one block tile)
    for path in (0, 1):
        with G.tuning(factgrass_path=path):
            st = torch.zeros(1, dtype=torch.int32, device="cuda")
            out = torch.full((cfg.B, cfg.k), 5.0, device="cuda")
            G.factgrass_compress(A, Gt, _dev_mask(G, mi), _dev_mask(G, mo), cfg.k, cfg.s, seed, out=out, dev_status=st)
            torch.cuda.synchronize()
            assert int(st.item()) == 0
        rel = max(rel, check_close(out.cpu().numpy(), ref, absum, TOL_F32 if f32 else TOL_BF16, chain, eps=EPS_TC,
                                   what=f"factgrass path {path} {lay} B={cfg.B} T={cfg.T} k'={cfg.kin}x{cfg.kout} "
                                        f"k={cfg.k} {dtype}"))
    return rel


@pytest.mark.parametrize("kw", [
    dict(),                                                          # odd sizes, one 64x64 tile
    dict(kin=5, kout=4, k=7, T=1),                                   # one token, tiny block
    dict(kin=64, kout=64, k=1024, T=200, B=4),                       # configs 4/5 tile, ragged token tail
    dict(kin=96, kout=160, k=4096, T=33),                            # mask = every coordinate; 128 tile; 2 column tiles
    dict(layers=None, kin=128, kout=128, k=4096, T=130, B=3),        # config 3 tile
    dict(layers=None, kin=130, kout=260, k=5000, T=64, B=2),         # several block tiles in both directions
    dict(kin=24, kout=40, k=50_000, T=40),                           # k too large for shared-memory bins
    dict(kin=24, kout=40, k=97, s=2),                                # two draws per position
    dict(kin=64, kout=64, k=256, T=300, pad_frac=0.2, g_dist="laplace"),
])
def test_factgrass_parity(G, W, oracle_mod, kw):
    kw = dict(kw)
    if "layers" in kw and kw["layers"] is None:
        kw["layers"] = (W.LinearLayer("l", 768, 3072),)
    _fact_case(G, W, oracle_mod, _fact_cfg(W, **kw))


@pytest.mark.parametrize("kw", [
    dict(),
    dict(kin=64, kout=64, k=1024, T=200, B=4),
    dict(layers=None, kin=128, kout=128, k=4096, T=130, B=3),
    dict(layers=None, kin=130, kout=260, k=5000, T=64, B=2),
    dict(kin=24, kout=40, k=97, s=2),
    dict(kin=64, kout=64, k=256, T=300, pad_frac=0.2, g_dist="laplace"),
])
def test_factgrass_fp32_inputs(G, W, oracle_mod, kw):
    """fp32 factors: the contraction runs on exact bf16 splits and must hold the fp32 tolerance."""
    kw = dict(kw)
    if "layers" in kw and kw["layers"] is None:
        kw["layers"] = (W.LinearLayer("l", 768, 3072),)
    rel = _fact_case(G, W, oracle_mod, _fact_cfg(W, **kw), dtype=torch.float32)
    assert rel < 1e-4


def test_factgrass_fp32_tile128(G, W, oracle_mod, tune):
    tune(factgrass_tile=128)
    cfg = _fact_cfg(W, layers=(W.LinearLayer("l", 768, 3072),), kin=128, kout=128, k=4096, T=130, B=3)
    _fact_case(G, W, oracle_mod, cfg, dtype=torch.float32)
    _fact_case(G, W, oracle_mod, cfg)


@pytest.mark.parametrize("chunk", [32, 64, 1 << 20])
def test_factgrass_token_chunking(G, W, oracle_mod, tune, chunk):
    """Splitting the token sum over CTAs (linearity of SJLT) does not change the result."""
    tune(factgrass_chunk=chunk)
    _fact_case(G, W, oracle_mod, _fact_cfg(W, T=250, kin=64, kout=64, k=512))


@pytest.mark.parametrize("tile", [64, 128])
def test_factgrass_seeded_shape_sweep(G, W, oracle_mod, tune, tile):
    """Seeded random shapes: layer widths, mask sizes around the 64 / 128 tile edges, token counts that end inside a
    32-token stage, output lengths on both sides of the block size, one or two draws, bf16 and fp32 factors."""
    tune(factgrass_tile=tile)
    rng = np.random.default_rng(1234 + tile)
    for case in range(10):
        d_in, d_out = int(rng.integers(8, 700)), int(rng.integers(8, 700))
        kin = int(min(d_in, rng.choice([1, 7, 63, 64, 65, 127, 128, 129, 200])))
        kout = int(min(d_out, rng.choice([1, 9, 63, 64, 65, 127, 128, 129, 150])))
        cfg = _fact_cfg(W, layers=(W.LinearLayer("l", d_in, d_out),), B=int(rng.integers(1, 5)),
                        T=int(rng.integers(1, 260)), kin=kin, kout=kout, k=int(rng.integers(1, 3 * kin * kout + 2)),
                        s=int(rng.choice([1, 1, 2])), data_seed=300 + case, mask_seed=case, hash_seed=5 * case + 1)
        _fact_case(G, W, oracle_mod, cfg, dtype=torch.float32 if case % 3 == 2 else torch.bfloat16)


def test_factgrass_scaled_configs(G, W, oracle_mod):
    c3 = dataclasses.replace(W.CONFIG3, B=4, T=256)
    _fact_case(G, W, oracle_mod, c3)
    c4 = dataclasses.replace(W.CONFIG4, B=2, T=256)
    for l in (0, 1, 3):
        _fact_case(G, W, oracle_mod, c4, l=l)
    c5 = dataclasses.replace(W.CONFIG5, B=1, T=256)
    for l in (1, 4, 6):
        _fact_case(G, W, oracle_mod, c5, l=l)


def test_factgrass_padding_tokens_change_nothing(G, W, oracle_mod, fg_path):
    cfg = _fact_cfg(W, T=64, kin=64, kout=64, k=512)
    A, Gt = W.layer_io(cfg, 0, device="cuda")
    mi = _dev_mask(G, oracle_mod.random_mask(96, 64, 1))
    mo = _dev_mask(G, oracle_mod.random_mask(160, 64, 2))
    a = G.factgrass_compress(A, Gt, mi, mo, 512, 1, 9)
    A2 = torch.cat([A, torch.randn_like(A)], dim=1).contiguous()
    G2 = torch.cat([Gt, torch.zeros_like(Gt)], dim=1).contiguous()
    b = G.factgrass_compress(A2, G2, mi, mo, 512, 1, 9)
    # same sums, possibly split over different token chunks: equal up to fp32 rounding order
    scale = float(a.abs().max())
    assert float((a - b).abs().max()) <= 1e-5 * scale


def test_factgrass_errors_and_empty(G, W, oracle_mod):
    cfg = _fact_cfg(W)
    A, Gt = W.layer_io(cfg, 0, device="cuda")
    mi = oracle_mod.random_mask(96, 24, 1)
    mo = oracle_mod.random_mask(160, 40, 2)
    # T = 0: zero output
    o = torch.full((3, 97), 5.0, device="cuda")
    G.factgrass_compress(A[:, :0].contiguous(), Gt[:, :0].contiguous(), _dev_mask(G, mi), _dev_mask(G, mo), 97, 1, 0, out=o)
    assert torch.all(o == 0)
    # A and G must have the same dtype
    with pytest.raises((G.GrassError, AssertionError, TypeError)):
        G.factgrass_compress(A.float(), Gt, _dev_mask(G, mi), _dev_mask(G, mo), 97, 1, 0)
    # an out-of-range mask index is skipped and flagged
    bad = mo.copy()
    bad[-1] = 4_000_000_000
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    got = G.factgrass_compress(A, Gt, _dev_mask(G, mi), _dev_mask(G, bad), 97, 1, 0, dev_status=st).cpu().numpy()
    assert int(st.item()) & 1
    G0 = Gt.clone()
    G0[:, :, int(mo[-1])] = 0
    ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(G0), mi, mo, 97, 1, 0)
    check_close(got, ref, absum, TOL_BF16, cfg.T + 64, eps=EPS_TC, what="bad factor index skipped")


# ------------------------------------------------------------------ grouped

def _group(G, W, oracle_mod, cfg, layer_ids, offsets=None):
    layers, refs = [], []
    off = 0
    for n, l in enumerate(layer_ids):
        lay = cfg.layers[l]
        A, Gt = W.layer_io(cfg, l, device="cuda")
        s_in, s_out = W.layer_mask_seeds(cfg, l)
        mi = oracle_mod.random_mask(lay.d_in, cfg.kin, s_in)
        mo = oracle_mod.random_mask(lay.d_out, cfg.kout, s_out)
        o = off if offsets is None else offsets[n]
        layers.append(dict(A=A, G=Gt, mask_in=_dev_mask(G, mi), mask_out=_dev_mask(G, mo), k=cfg.k, s=cfg.s,
                           seed=W.layer_hash_seed(cfg, l), out_offset=o))
        refs.append((o, mi, mo, W.layer_hash_seed(cfg, l), A, Gt))
        off += cfg.k
    return layers, refs


def test_factgrass_grouped_parity(G, W, oracle_mod, fg_path):
    cfg = dataclasses.replace(W.CONFIG4, B=3, T=96, layers=W.CONFIG4.layers[:8])
    ids = list(range(8))
    layers, refs = _group(G, W, oracle_mod, cfg, ids)
    group = G.GroupedLayers(layers)
    ld = cfg.k * len(ids) + 5
    out = torch.full((cfg.B, ld), 3.0, device="cuda")
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(len(ids)), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    G.factgrass_compress_grouped(group, out, ws, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    host = out.cpu().numpy()
    assert np.all(host[:, cfg.k * len(ids):] == 3.0)            # columns outside every layer's range untouched
    for (o, mi, mo, seed, A, Gt) in refs:
        ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, cfg.k, cfg.s, seed)
        check_close(host[:, o:o + cfg.k], ref, absum, TOL_BF16, cfg.T + 64, eps=EPS_TC, what=f"grouped off={o}")
        single = G.factgrass_compress(A, Gt, _dev_mask(G, mi), _dev_mask(G, mo), cfg.k, cfg.s, seed).cpu().numpy()
        check_close(single, ref, absum, TOL_BF16, cfg.T + 64, eps=EPS_TC, what="single")


def test_factgrass_grouped_mixed_layers(G, W, oracle_mod, fg_path):
    """Layers of one call may differ in d_in/d_out, mask sizes, k, s and seed."""
    B, T = 2, 50
    specs = [(96, 160, 24, 40, 97, 1), (200, 64, 64, 64, 1024, 1), (768, 3072, 100, 130, 300, 2)]
    layers, refs, off = [], [], 0
    for n, (d_in, d_out, kin, kout, k, s) in enumerate(specs):
        cfg = _fact_cfg(W, layers=(W.LinearLayer("x", d_in, d_out),), B=B, T=T, kin=kin, kout=kout, k=k, s=s,
                        data_seed=100 + n)
        A, Gt = W.layer_io(cfg, 0, device="cuda")
        mi = oracle_mod.random_mask(d_in, kin, n)
        mo = oracle_mod.random_mask(d_out, kout, n + 50)
        layers.append(dict(A=A, G=Gt, mask_in=_dev_mask(G, mi), mask_out=_dev_mask(G, mo), k=k, s=s, seed=n * 3,
                           out_offset=off))
        refs.append((off, k, s, n * 3, mi, mo, A, Gt))
        off += k + 3
    out = torch.zeros(B, off, device="cuda")
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(len(specs)), dtype=torch.uint8, device="cuda")
    G.factgrass_compress_grouped(G.GroupedLayers(layers), out, ws)
    host = out.cpu().numpy()
    for (o, k, s, seed, mi, mo, A, Gt) in refs:
        ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, k, s, seed)
        check_close(host[:, o:o + k], ref, absum, TOL_BF16, T + 64, eps=EPS_TC, what=f"mixed off={o}")


def test_factgrass_grouped_layer_with_an_empty_mask(G, W, oracle_mod, fg_path):
    """A layer whose input-factor mask is empty has no block: its output range must come back as zeros, the
    other layers must be untouched by it, and no device fault may be flagged."""
    B, T = 2, 70
    specs = [(96, 160, 24, 40, 97), (200, 64, 0, 64, 128), (128, 128, 64, 0, 64), (768, 3072, 64, 64, 300)]
    layers, refs, off = [], [], 0
    for n, (d_in, d_out, kin, kout, k) in enumerate(specs):
        cfg = _fact_cfg(W, layers=(W.LinearLayer("x", d_in, d_out),), B=B, T=T, kin=max(kin, 1), kout=max(kout, 1),
                        k=k, data_seed=200 + n)
        A, Gt = W.layer_io(cfg, 0, device="cuda")
        mi = oracle_mod.random_mask(d_in, kin, n) if kin else np.empty(0, dtype=np.uint32)
        mo = oracle_mod.random_mask(d_out, kout, n + 50) if kout else np.empty(0, dtype=np.uint32)
        layers.append(dict(A=A, G=Gt, mask_in=_dev_mask(G, mi), mask_out=_dev_mask(G, mo), k=k, s=1, seed=n,
                           out_offset=off))
        refs.append((off, k, n, mi, mo, A, Gt))
        off += k
    out = torch.full((B, off), 7.0, device="cuda")
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(len(specs)), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    G.factgrass_compress_grouped(G.GroupedLayers(layers), out, ws, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    host = out.cpu().numpy()
    for (o, k, seed, mi, mo, A, Gt) in refs:
        if mi.size == 0 or mo.size == 0:
            assert np.all(host[:, o:o + k] == 0.0)
            continue
        ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, k, 1, seed)
        check_close(host[:, o:o + k], ref, absum, TOL_BF16, T + 64, eps=EPS_TC, what=f"empty-mask group off={o}")


# ------------------------------------------------------------------ grass_score

@pytest.mark.parametrize("N,M,D", [(300, 70, 257), (128, 128, 64), (1, 1, 1), (513, 256, 4096), (5, 3, 10),
                                   (300, 70, 260), (200, 24, 96), (130, 300, 64), (1, 1, 4), (257, 8, 36)])
def test_grass_score_parity(G, W, oracle_mod, N, M, D):
    tr, te = W.score_vectors(N, M, D, 31, device="cuda")
    sc = G.grass_score(tr, te).cpu().numpy()
    ref, absum = oracle_mod.score(tr.cpu().numpy(), te.cpu().numpy())
    check_close(sc, ref, absum, TOL_F32, D + 8, what=f"score {N}x{M}x{D}")


def test_grass_score_many_aligned_shapes(G, W, oracle_mod):
    """Seeded sweep over shapes that take the tensor-core path (row strides a multiple of four floats): row
    counts around the 128 / 256 tile edges, several column tiles, k extents that end inside a 32-wide k tile,
    and operands that are column slices of wider matrices."""
    rng = np.random.default_rng(77)
    shapes = [(127, 255, 28), (129, 257, 36), (255, 1, 4), (256, 256, 32), (257, 513, 100), (384, 16, 2052),
              (1, 300, 64), (640, 40, 8)]
    shapes += [(int(rng.integers(1, 700)), int(rng.integers(1, 600)), 4 * int(rng.integers(1, 300))) for _ in range(6)]
    for (N, M, D) in shapes:
        pad = 4 * int(rng.integers(0, 3))
        trw, tew = W.score_vectors(N, M, D + pad, 900 + N, device="cuda")
        tr, te = trw[:, :D], tew[:, :D]
        sc = G.grass_score(tr, te).cpu().numpy()
        ref, absum = oracle_mod.score(np.ascontiguousarray(tr.cpu().numpy()), np.ascontiguousarray(te.cpu().numpy()))
        check_close(sc, ref, absum, TOL_F32, D + 8, what=f"score {N}x{M}x{D} ld={D + pad}")


def test_grass_score_strided_and_compressed_inputs(G, W, oracle_mod):
    """Scores of actual compressed gradients; train rows taken from a wider matrix."""
    g = W.dense_gradients(40, 30_000, 0.7, "normal", 1.0, 9, device="cuda")
    idx = _dev_mask(G, oracle_mod.random_mask(30_000, 6_000, 0))
    comp = G.grass_compress(g, idx, 510, 1, 4)
    wide = torch.zeros(40, 520, device="cuda")
    wide[:, :510] = comp
    tr, te = wide[:30, :510], comp[30:]
    sc = G.grass_score(tr, te).cpu().numpy()
    ref, absum = oracle_mod.score(np.ascontiguousarray(tr.cpu().numpy()), np.ascontiguousarray(te.cpu().numpy()))
    check_close(sc, ref, absum, TOL_F32, 520, what="score of compressed")


def test_grass_score_split_contraction(G, W, oracle_mod, tune):
    """The contraction split over several CTAs per output tile (partial products added into the zeroed output):
    forced through the tuning hook, with a ragged last split, vector and scalar reductions (output row
    stride a multiple of four floats or not), stale data in the output buffer; then the two automatic cases,
    a long contraction (D > 16,384) and a small output that would leave most SMs idle."""
    for splits, (N, M, D), ld_s in [(3, (300, 70, 260), 70), (5, (129, 257, 1000), 260), (2, (256, 256, 64), 256),
                                    (64, (40, 300, 128), 301), (7, (513, 24, 4096), 24)]:
        tune(score_splits=splits)
        tr, te = W.score_vectors(N, M, D, 55 + splits, device="cuda")
        buf = torch.full((N, ld_s), 123.0, device="cuda")
        sc = G.grass_score(tr, te, out=buf[:, :M])
        ref, absum = oracle_mod.score(tr.cpu().numpy(), te.cpu().numpy())
        check_close(sc.cpu().numpy(), ref, absum, TOL_F32, D + 8 + splits, what=f"score {N}x{M}x{D}, {splits} splits")
        if ld_s > M:
            assert torch.all(buf[:, M:] == 123.0), "columns beyond M must not be touched"
    tune(score_splits=None)
    for (N, M, D) in [(200, 100, 20_000), (64, 32, 8_192), (300, 520, 3_000)]:
        tr, te = W.score_vectors(N, M, D, 77, device="cuda")
        sc = G.grass_score(tr, te, out=torch.full((N, M), -5.0, device="cuda"))
        ref, absum = oracle_mod.score(tr.cpu().numpy(), te.cpu().numpy())
        check_close(sc.cpu().numpy(), ref, absum, TOL_F32, D + 64, what=f"score {N}x{M}x{D}, automatic split")


def test_grass_score_long_contraction_keeps_relative_accuracy(G, oracle_mod):
    """Positive operands, D = 262,144: nothing cancels, so every score must be right to 1e-4 relative.  The
    tensor core truncates its fp32 accumulator after every MMA; a single accumulator over 16,384 MMAs would be
    biased by several 1e-4, which is why long contractions are split into runs of 8,192 k-values."""
    N, M, D = 256, 64, 262_144
    g = torch.Generator(device="cuda")
    g.manual_seed(12)
    tr = torch.rand((N, D), generator=g, device="cuda") + 0.5
    te = torch.rand((M, D), generator=g, device="cuda") + 0.5
    sc = G.grass_score(tr, te).cpu().numpy().astype(np.float64)
    ref, _ = oracle_mod.score(tr.cpu().numpy(), te.cpu().numpy())
    rel = np.abs(sc - ref) / np.abs(ref)
    assert rel.max() <= 1e-4, rel.max()
