"""GPU parity of the host-buffer calls (inputs in pinned host memory): the staged path, which copies the inputs
to the device, and the in-place path, where the kernels gather from the host buffers directly."""
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


def _pinned(t):
    return torch.empty(t.shape, dtype=t.dtype, pin_memory=True).copy_(t)


@pytest.mark.parametrize("zero_copy", [False, True, None])
def test_grass_compress_host(G, W, oracle_mod, zero_copy):
    from paper_2505_18976_b200 import host_api
    p, kp, k, seed = 50_000, 3_000, 700, 11
    idx = oracle_mod.random_mask(p, kp, 3)
    chunks = [_pinned(W.dense_gradients(r, p, 0.6, "normal", 1.0, 20 + i, device="cpu")) for i, r in enumerate((5, 9, 2))]
    out = host_api.grass_compress_host(chunks, idx, k, 1, seed, zero_copy=zero_copy)
    assert out.shape == (16, k) and not out.is_cuda
    ob, _ = oracle_mod.sjlt_table(k, 1, seed, kp)
    row = 0
    for c in chunks:
        ref, absum = oracle_mod.grass(W.bits_of(c), idx, k, 1, seed)
        check_close(out[row:row + c.shape[0]].numpy(), ref, absum, TOL_F32, max_bin_load(ob, k) + 16,
                    what=f"host chunk at row {row}, zero_copy={zero_copy}")
        row += c.shape[0]


def test_grass_compress_binding_reads_pinned_bf16_rows_in_place(G, W, oracle_mod):
    p, kp, k, seed = 20_000, 1_500, 256, 5
    idx = oracle_mod.random_mask(p, kp, 9)
    g = _pinned(W.dense_gradients(7, p, 0.5, "normal", 1.0, 31, device="cpu").to(torch.bfloat16))
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = G.grass_compress(g, G.mask_to_device(idx), k, 2, seed, dev_status=st)
    assert out.is_cuda and int(st.item()) == 0
    ref, absum = oracle_mod.grass(W.bits_of(g), idx, k, 2, seed, dtype="bf16")
    check_close(out.cpu().numpy(), ref, absum, TOL_BF16, 64, what="pinned bf16 rows")


@pytest.mark.parametrize("zero_copy", [False, True, None])
def test_factgrass_compress_host(G, W, oracle_mod, zero_copy):
    from paper_2505_18976_b200 import host_api
    Bsz, T, k = 3, 150, 512
    gen = torch.Generator().manual_seed(77)
    shapes = [(96, 200), (200, 64), (128, 128)]
    groups, refs, off = [], [], 0
    for gi in range(2):
        grp = []
        for li, (d_in, d_out) in enumerate(shapes[gi:gi + 2]):
            A = _pinned(torch.randn((Bsz, T, d_in), generator=gen).to(torch.bfloat16))
            Gt = _pinned((torch.randn((Bsz, T, d_out), generator=gen) * 1e-2).to(torch.bfloat16))
            mi = oracle_mod.random_mask(d_in, 40, 100 + off)
            mo = oracle_mod.random_mask(d_out, 24, 200 + off)
            seed = 900 + off
            grp.append(dict(A=A, G=Gt, mask_in=mi, mask_out=mo, k=k, s=1, seed=seed, out_offset=off))
            refs.append((off, A, Gt, mi, mo, seed))
            off += k
        groups.append(grp)
    out = host_api.factgrass_compress_host(groups, Bsz, T, off, zero_copy=zero_copy)
    assert out.shape == (Bsz, off) and not out.is_cuda
    for (o, A, Gt, mi, mo, seed) in refs:
        ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, k, 1, seed)
        check_close(out[:, o:o + k].numpy(), ref, absum, TOL_BF16, T + 64, eps=EPS_TC,
                    what=f"host layer at offset {o}, zero_copy={zero_copy}")


def test_unpinned_host_input_is_refused(G):
    g = torch.zeros((2, 64))
    with pytest.raises(ValueError):
        G.grass_compress(g, None, 8, 1, 0, out=torch.empty((2, 8), device="cuda"))


def test_grass_score_host(G, W, oracle_mod):
    from paper_2505_18976_b200 import host_api
    tr, te = W.score_vectors(70, 20, 132, 3, device="cpu")
    sc = host_api.grass_score_host(_pinned(tr), _pinned(te))
    ref, absum = oracle_mod.score(tr.numpy(), te.numpy())
    check_close(sc.numpy(), ref, absum, TOL_F32, 140, what="host score")


def test_config4_block_in_place_matches_device_resident(G, W, oracle_mod):
    """One GPT-2-small block of config 4 (4 layers, 16 x 1,024 tokens) gathered from pinned host memory: same
    results as from device memory up to the order of the atomic adds, and parity with the oracle on one layer."""
    from paper_2505_18976_b200 import host_api
    c = W.CONFIG4
    dev_layers, host_layers = [], []
    for l in range(4):
        A, Gt = W.layer_io(c, l, device="cuda")
        s_in, s_out = W.layer_mask_seeds(c, l)
        mi = G.grass_random_mask_host(c.layers[l].d_in, c.kin, s_in)
        mo = G.grass_random_mask_host(c.layers[l].d_out, c.kout, s_out)
        common = dict(k=c.k, s=c.s, seed=W.layer_hash_seed(c, l), out_offset=l * c.k)
        dev_layers.append(dict(A=A, G=Gt, mask_in=G.mask_to_device(mi), mask_out=G.mask_to_device(mo), **common))
        host_layers.append(dict(A=_pinned(A.cpu()), G=_pinned(Gt.cpu()), mask_in=mi, mask_out=mo, **common))
    assert host_api.factgrass_in_place([host_layers])
    # the choice is made tensor by tensor: the 768-wide factors (three in four pieces touched) are copied, the
    # 2,304- and 3,072-wide ones are gathered in place
    plan, moved = host_api.factgrass_host_plan([host_layers])
    flat = [d for pair in plan for d in pair]
    assert True in flat and False in flat
    assert moved < sum(l["A"].numel() * 2 + l["G"].numel() * 2 for l in host_layers)
    out_dev = torch.empty((c.B, 4 * c.k), device="cuda")
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(4), dtype=torch.uint8, device="cuda")
    G.factgrass_compress_grouped(G.GroupedLayers(dev_layers), out_dev, ws)
    out_host = host_api.factgrass_compress_host([host_layers], c.B, c.T, 4 * c.k)
    a, b = out_dev.cpu().numpy().astype(np.float64), out_host.numpy().astype(np.float64)
    assert np.abs(a - b).max() <= 1e-5 * np.abs(a).max()
    l = 2
    ref, absum = oracle_mod.factgrass(W.bits_of(dev_layers[l]["A"]), W.bits_of(dev_layers[l]["G"]),
                                      host_layers[l]["mask_in"], host_layers[l]["mask_out"], c.k, c.s,
                                      W.layer_hash_seed(c, l))
    check_close(b[:, l * c.k:(l + 1) * c.k], ref, absum, TOL_BF16, c.T + 64, eps=EPS_TC, what="config 4 block, in place")


def test_single_layer_and_mask_calls_read_pinned_inputs_in_place(G, W, oracle_mod):
    """factgrass_compress, factmask_compress and grass_mask given pinned host tensors."""
    gen = torch.Generator().manual_seed(5)
    A = _pinned(torch.randn((2, 90, 200), generator=gen).to(torch.bfloat16))
    Gt = _pinned((torch.randn((2, 90, 120), generator=gen) * 1e-2).to(torch.bfloat16))
    mi, mo = oracle_mod.random_mask(200, 30, 1), oracle_mod.random_mask(120, 20, 2)
    dmi, dmo = G.mask_to_device(mi), G.mask_to_device(mo)
    out = G.factgrass_compress(A, Gt, dmi, dmo, 333, 1, 17)
    assert out.is_cuda
    ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, 333, 1, 17)
    check_close(out.cpu().numpy(), ref, absum, TOL_BF16, 90 + 64, eps=EPS_TC, what="pinned single layer")
    blk = G.factmask_compress(A, Gt, dmi, dmo)
    ref, absum = oracle_mod.factmask(W.bits_of(A), W.bits_of(Gt), mi, mo)
    check_close(blk.cpu().numpy(), ref, absum, TOL_BF16, 90 + 8, eps=EPS_TC, what="pinned factorised mask")
    g = _pinned(W.dense_gradients(3, 5_000, 0.5, "normal", 1.0, 8, device="cpu"))
    idx = oracle_mod.random_mask(5_000, 400, 3)
    mk = G.grass_mask(g, G.mask_to_device(idx))
    assert np.array_equal(mk.cpu().numpy(), oracle_mod.mask(W.bits_of(g), idx))
