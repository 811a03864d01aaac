"""GPU parity at the full benchmark sizes, in the launch configuration the benchmark times.

Every configuration is run exactly as ``bench.py`` runs it (same workload generators, same
calls, whole batch / all layers in one launch).  Where the CPU oracle can do the whole output in
seconds (configs 1 and 3) every element is compared; otherwise the outputs of a sample of rows
or layers are recomputed by the oracle from the same bytes, and the rest is checked by
properties that hold at any size (finite, untouched neighbours, mass that matches the input).
"""
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


@pytest.fixture(autouse=True)
def _release_memory():
    yield
    torch.cuda.synchronize()
    torch.cuda.empty_cache()


def test_config1_full_every_output(G, W, oracle_mod):
    c = W.CONFIG1
    g = W.dense_gradients(c.batch, c.p, c.zero_prob, c.dist, c.scale, c.data_seed, device="cuda")
    idx = G.grass_random_mask_host(c.p, c.kprime, c.mask_seed)
    assert np.array_equal(idx, oracle_mod.random_mask(c.p, c.kprime, c.mask_seed))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = G.grass_compress(g, G.mask_to_device(idx), c.k, c.s, c.hash_seed, dev_status=st)
    assert int(st.item()) == 0
    ref, absum = oracle_mod.grass(W.bits_of(g), idx, c.k, c.s, c.hash_seed)
    ob, _ = oracle_mod.sjlt_table(c.k, c.s, c.hash_seed, c.kprime)
    check_close(out.cpu().numpy(), ref, absum, TOL_F32, max_bin_load(ob, c.k) + 16, what="config 1 full")


def test_config2_full_batch_sampled_rows(G, W, oracle_mod):
    """One batch of 512 x 4,194,304 fp32 (8.6 GB) through one call; the oracle recomputes 24 rows."""
    c = W.CONFIG2
    g = W.dense_gradients(c.batch, c.p, c.zero_prob, c.dist, c.scale, c.data_seed, device="cuda")
    idx = G.grass_random_mask_host(c.p, c.kprime, c.mask_seed)
    assert np.array_equal(idx, oracle_mod.random_mask(c.p, c.kprime, c.mask_seed))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    wide = torch.full((c.batch, c.k + 3), 9.0, device="cuda")              # a strided output with a guard band
    out = wide[:, :c.k]
    G.grass_compress(g, G.mask_to_device(idx), c.k, c.s, c.hash_seed, out=out, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    rows = sorted(set([0, 1, 255, 256, 510, 511] + list(np.random.default_rng(2).integers(0, c.batch, 18))))
    sample = g[rows].cpu().numpy()
    ref, absum = oracle_mod.grass(sample, idx, c.k, c.s, c.hash_seed)
    ob, _ = oracle_mod.sjlt_table(c.k, c.s, c.hash_seed, c.kprime)
    host = out.cpu().numpy()
    check_close(host[rows], ref, absum, TOL_F32, max_bin_load(ob, c.k) + 16, what="config 2 sampled rows")
    # every row: finite, and the signed total of a row equals the signed total of its masked entries
    assert np.isfinite(host).all()
    didx = G.mask_to_device(idx).long()
    sign = torch.from_numpy(oracle_mod.sjlt_table(c.k, c.s, c.hash_seed, c.kprime)[1].astype(np.float64)).cuda()
    tot_ref = torch.zeros(c.batch, dtype=torch.float64, device="cuda")
    mass = torch.zeros(c.batch, dtype=torch.float64, device="cuda")
    for r0 in range(0, c.batch, 64):
        gm = g[r0:r0 + 64].index_select(1, didx).double()
        tot_ref[r0:r0 + 64] = (gm * sign).sum(1)
        mass[r0:r0 + 64] = gm.abs().sum(1)
    tot = out.double().sum(1)
    assert torch.all((tot - tot_ref).abs() <= 1e-5 * mass)
    assert torch.all(wide[:, c.k:] == 9.0)


def test_config3_full_every_output(G, W, oracle_mod, fg_path):
    c = W.CONFIG3
    lay = c.layers[0]
    A, Gt = W.layer_io(c, 0, device="cuda")
    s_in, s_out = W.layer_mask_seeds(c, 0)
    mi = G.grass_random_mask_host(lay.d_in, c.kin, s_in)
    mo = G.grass_random_mask_host(lay.d_out, c.kout, s_out)
    seed = W.layer_hash_seed(c, 0)
    layers = [dict(A=A, G=Gt, mask_in=G.mask_to_device(mi), mask_out=G.mask_to_device(mo), k=c.k, s=c.s, seed=seed,
                   out_offset=0)]
    out = torch.empty(c.B, c.k, device="cuda")
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(1), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    G.factgrass_compress_grouped(G.GroupedLayers(layers), out, ws, dev_status=st)
    assert int(st.item()) == 0
    ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, c.k, c.s, seed)
    ob, _ = oracle_mod.sjlt_table(c.k, c.s, seed, c.kin * c.kout)
    check_close(out.cpu().numpy(), ref, absum, TOL_BF16, c.T + max_bin_load(ob, c.k) + 64, eps=EPS_TC,
                what="config 3 full")


def _grouped_full(G, W, oracle_mod, c, sample_layers, what):
    layers, keep = [], {}
    for l, lay in enumerate(c.layers):
        A, Gt = W.layer_io(c, l, device="cuda")
        s_in, s_out = W.layer_mask_seeds(c, l)
        mi = G.grass_random_mask_host(lay.d_in, c.kin, s_in)
        mo = G.grass_random_mask_host(lay.d_out, c.kout, s_out)
        layers.append(dict(A=A, G=Gt, mask_in=G.mask_to_device(mi), mask_out=G.mask_to_device(mo), k=c.k, s=c.s,
                           seed=W.layer_hash_seed(c, l), out_offset=l * c.k))
        if l in sample_layers:
            keep[l] = (mi, mo)
    out = torch.full((c.B, c.out_dim), float("nan"), device="cuda")
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(len(layers)), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    G.factgrass_compress_grouped(G.GroupedLayers(layers), out, ws, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    host = out.cpu().numpy()
    assert np.isfinite(host).all()                       # every layer's range was written
    per_layer_mass = np.abs(host).reshape(c.B, len(c.layers), c.k).sum(2)
    assert (per_layer_mass > 0).all()
    for l in sorted(sample_layers):
        mi, mo = keep[l]
        seed = W.layer_hash_seed(c, l)
        assert np.array_equal(mi, oracle_mod.random_mask(c.layers[l].d_in, c.kin, W.layer_mask_seeds(c, l)[0]))
        ref, absum = oracle_mod.factgrass(W.bits_of(layers[l]["A"]), W.bits_of(layers[l]["G"]), mi, mo, c.k, c.s, seed)
        ob, _ = oracle_mod.sjlt_table(c.k, c.s, seed, c.kin * c.kout)
        check_close(host[:, l * c.k:(l + 1) * c.k], ref, absum, TOL_BF16, c.T + max_bin_load(ob, c.k) + 64,
                    eps=EPS_TC, what=f"{what} layer {l} ({c.layers[l].name})")
    return out


def test_config4_full_all_layers_one_launch(G, W, oracle_mod):
    """48 layers x 16 x 1,024 tokens in one grouped launch; the oracle recomputes 12 of the layers."""
    _grouped_full(G, W, oracle_mod, W.CONFIG4, {0, 1, 2, 3, 9, 14, 20, 27, 33, 38, 46, 47}, "config 4")


def test_config5_full_all_layers_one_launch_and_score(G, W, oracle_mod):
    """224 layers x 4 x 2,048 tokens (42.9 GB resident) in one grouped launch; the oracle recomputes 10 layers,
    one of every shape among them; then the full-size score with 256 sampled train rows."""
    free, _ = torch.cuda.mem_get_info()
    if free < 60 * 2 ** 30:
        pytest.skip("needs about 50 GB of free device memory")
    c = W.CONFIG5
    _grouped_full(G, W, oracle_mod, c, {0, 1, 2, 3, 4, 5, 6, 108, 117, 223}, "config 5")
    torch.cuda.empty_cache()
    tr, te = W.score_vectors(c.score_n_train, c.score_n_test, c.k, c.data_seed + 7, device="cuda")
    sc = G.grass_score(tr, te)
    rows = sorted(set([0, 127, 128, 16_383] + list(np.random.default_rng(5).integers(0, c.score_n_train, 252))))
    ref, absum = oracle_mod.score(tr[rows].cpu().numpy(), te.cpu().numpy())
    check_close(sc[rows].cpu().numpy(), ref, absum, TOL_F32, c.k + 8, what="config 5 score, sampled train rows")
    # all rows: Cauchy-Schwarz and the row sum <train_i, sum_m test_m>
    assert torch.isfinite(sc).all()
    bound = tr.double().norm(dim=1)[:, None] * te.double().norm(dim=1)[None, :]
    assert torch.all(sc.double().abs() <= bound * (1 + 1e-6))
    rowsum = tr.double() @ te.double().sum(0)
    absrow = tr.double().abs() @ te.double().abs().sum(0)
    assert torch.all((sc.double().sum(1) - rowsum).abs() <= 1e-5 * absrow)


def test_grass_compress_row_longer_than_2_to_31(G, oracle_mod):
    """One bf16 row of 3 * 10^9 entries (6 GB): index arithmetic beyond 32 bits.  The oracle works on the
    gathered entries with the identity mask, which is the same thing by definition (the hash argument is the
    position in the masked vector)."""
    p, kp, k, seed = 3_000_000_000, 20_000, 1_024, 41
    g = torch.zeros((1, p), dtype=torch.bfloat16, device="cuda")
    rng = np.random.default_rng(3)
    idx = np.unique(np.concatenate([rng.integers(0, p, kp - 3, dtype=np.int64), [0, 2 ** 31 + 5, p - 1]]))
    idx = idx[idx != 12345].astype(np.uint32)
    vals = torch.randn(idx.size, device="cuda").to(torch.bfloat16)
    g[0, torch.from_numpy(idx.astype(np.int64)).cuda()] = vals
    g[0, 12345] = 7.0                                   # an entry outside the mask must not be read into the result
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = G.grass_compress(g, G.mask_to_device(idx), k, 1, seed, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    gathered = vals.view(torch.uint16).cpu().numpy().reshape(1, -1)
    ref, absum = oracle_mod.grass(np.ascontiguousarray(gathered), None, k, 1, seed, dtype="bf16")
    check_close(out.cpu().numpy(), ref, absum, TOL_BF16, 64, what="row longer than 2^31")
    mk = G.grass_mask(g, G.mask_to_device(idx)).cpu().numpy()
    assert np.array_equal(mk[0], vals.float().cpu().numpy())


def test_factgrass_operand_larger_than_2_to_31_elements(G, W, oracle_mod):
    """A of 1 x 36,000 x 65,536 bf16 (2.36 * 10^9 elements): row offsets beyond 32 bits.  The oracle gets the
    gathered columns with identity masks (the same thing by definition)."""
    T, d_in, d_out, kin, kout, k, seed = 36_000, 65_536, 96, 64, 40, 777, 5
    gen = torch.Generator(device="cuda")
    gen.manual_seed(12)
    A = torch.empty((1, T, d_in), dtype=torch.bfloat16, device="cuda")
    for t0 in range(0, T, 4_000):
        A[0, t0:t0 + 4_000] = torch.randn((min(4_000, T - t0), d_in), generator=gen, device="cuda").to(torch.bfloat16)
    Gt = (torch.randn((1, T, d_out), generator=gen, device="cuda") * 1e-3).to(torch.bfloat16)
    mi = oracle_mod.random_mask(d_in, kin, 1)
    mo = oracle_mod.random_mask(d_out, kout, 2)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = G.factgrass_compress(A, Gt, G.mask_to_device(mi), G.mask_to_device(mo), k, 1, seed, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    Am = A[:, :, torch.from_numpy(mi.astype(np.int64)).cuda()].contiguous()
    Gm = Gt[:, :, torch.from_numpy(mo.astype(np.int64)).cuda()].contiguous()
    ref, absum = oracle_mod.factgrass(W.bits_of(Am), W.bits_of(Gm), np.arange(kin, dtype=np.uint32),
                                      np.arange(kout, dtype=np.uint32), k, 1, seed)
    check_close(out.cpu().numpy(), ref, absum, TOL_BF16, T + 64, eps=EPS_TC, what="operand larger than 2^31 elements")


def test_config5_score_over_the_full_concatenation(G, oracle_mod):
    """Scores over all 224 layers at once: train 16,384 x 917,504 fp32 (60 GB), test 256 x 917,504.  The oracle
    recomputes sampled train rows; every row is checked against the Cauchy-Schwarz bound and the row-sum identity."""
    free, _ = torch.cuda.mem_get_info()
    if free < 100 * 2 ** 30:
        pytest.skip("needs about 95 GB of free device memory")
    N, M, D = 16_384, 256, 224 * 4_096
    g = torch.Generator(device="cuda")
    g.manual_seed(2_005)
    tr = torch.empty((N, D), dtype=torch.float32, device="cuda")
    for i in range(0, N, 1_024):
        tr[i:i + 1_024].normal_(generator=g)
    te = torch.randn((M, D), generator=g, device="cuda")
    sc = G.grass_score(tr, te)
    torch.cuda.synchronize()
    assert torch.isfinite(sc).all()
    rows = [0, 127, 128, 255, 256, 8_191, 16_383] + [int(r) for r in np.random.default_rng(8).integers(0, N, 9)]
    ref, absum = oracle_mod.score(tr[rows].cpu().numpy(), te.cpu().numpy())
    check_close(sc[rows].cpu().numpy(), ref, absum, TOL_F32, 8_192 + 8 + 112, what="score over D = 917,504, sampled rows")
    te_sum, te_abs, te_norm = te.double().sum(0), te.double().abs().sum(0), te.double().norm(dim=1)
    for i in range(0, N, 2_048):
        blk = tr[i:i + 2_048].double()
        s = sc[i:i + 2_048].double()
        assert torch.all(s.abs() <= blk.norm(dim=1)[:, None] * te_norm[None, :] * (1 + 1e-6))
        assert torch.all((s.sum(1) - blk @ te_sum).abs() <= 1e-5 * (blk.abs() @ te_abs))
        del blk


def test_long_accumulations_keep_relative_accuracy(G, W, oracle_mod):
    """Positive data, so nothing cancels and every output must be right to 1e-4 relative: the projected FIM of
    400,000 samples at k = 2,048 (enough tiles that each would otherwise sum a third of the samples in one
    accumulator), and FactGraSS over 32,768 tokens for 1,024 (layer, sample) pairs.  Accumulators of the tensor
    core are truncated after every MMA, so no run may exceed 8,192 rows."""
    n, k = 400_000, 2_048
    g = torch.Generator(device="cuda")
    g.manual_seed(77)
    X = torch.rand((n, k), generator=g, device="cuda") + 0.5
    F = G.grass_fim(X)
    cols = [0, 1, 127, 128, 1_000, 2_047]
    ref, _ = oracle_mod.fim(np.ascontiguousarray(X[:, cols].cpu().numpy()))
    got = F[cols][:, cols].cpu().numpy().astype(np.float64)
    assert (np.abs(got - ref) / np.abs(ref)).max() <= 1e-4
    del X, F
    torch.cuda.empty_cache()

    B, T, d, kk, k_out, L = 256, 32_768, 64, 64, 4_096, 4
    A = (torch.rand((B, T, d), generator=g, device="cuda") + 0.5).to(torch.bfloat16)
    Gt = (torch.rand((B, T, d), generator=g, device="cuda") + 0.5).to(torch.bfloat16)
    ident = np.arange(kk, dtype=np.uint32)
    dev_ident = G.mask_to_device(ident)
    layers = [dict(A=A, G=Gt, mask_in=dev_ident, mask_out=dev_ident, k=k_out, s=1, seed=900 + l, out_offset=l * k_out)
              for l in range(L)]
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(L), dtype=torch.uint8, device="cuda")
    out = torch.empty((B, L * k_out), device="cuda")
    G.factgrass_compress_grouped(G.GroupedLayers(layers), out, ws)
    for (b, l) in [(0, 0), (255, 3)]:
        ref, absum = oracle_mod.factgrass(W.bits_of(A[b:b + 1]), W.bits_of(Gt[b:b + 1]), ident, ident, k_out, 1, 900 + l)
        got = out[b, l * k_out:(l + 1) * k_out].cpu().numpy().astype(np.float64)
        # a bin holds entries of both signs: compare against the sum of magnitudes
        used = absum[0] > 0
        assert (np.abs(got - ref[0])[used] / absum[0][used]).max() <= 1e-4
        assert np.all(got[~used] == 0.0)
