"""GPU parity of the stand-alone Mask compressors (Section 3.2) against the CPU oracle."""
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


@pytest.fixture(scope="module")
def W():
    from paper_2505_18976_b200 import workloads
    return workloads


@pytest.mark.parametrize("n,p,kp,dtype,ld", [(7, 10_007, 1_237, torch.float32, None), (3, 65_536, 8_192, torch.float32, None),
                                             (5, 9_001, 700, torch.float32, 9_016), (4, 50_000, 5_000, torch.bfloat16, None),
                                             (2, 300, 300, torch.float32, None)])
def test_grass_mask_bit_exact(G, W, oracle_mod, n, p, kp, dtype, ld):
    g = W.dense_gradients(n, p, 0.5, "normal", 1.0, 4, device="cuda", dtype=dtype, ld=ld)
    idx = oracle_mod.random_mask(p, kp, 9)
    out = G.grass_mask(g, G.mask_to_device(idx), p=p).cpu().numpy()
    ref = oracle_mod.mask(W.bits_of(g), idx, dtype="f32" if dtype == torch.float32 else "bf16", p=p)
    assert np.array_equal(out.astype(np.float64), ref)          # a gather: exact


def test_grass_mask_bad_index_and_errors(G, oracle_mod):
    g = torch.randn(2, 100, device="cuda")
    idx = oracle_mod.random_mask(100, 10, 1)
    bad = idx.copy()
    bad[-1] = 4_000_000_000
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = G.grass_mask(g, G.mask_to_device(bad), dev_status=st).cpu().numpy()
    assert int(st.item()) & 1 and np.all(out[:, -1] == 0)
    assert np.array_equal(out[:, :-1], g.cpu().numpy()[:, idx[:-1]])
    with pytest.raises(G.GrassError):
        G.grass_mask(g, G.mask_to_device(np.arange(101, dtype=np.uint32)))     # k' > p


@pytest.mark.parametrize("B,T,d_in,d_out,kin,kout,dtype", [
    (3, 70, 96, 160, 24, 40, torch.bfloat16), (4, 200, 768, 3072, 64, 64, torch.bfloat16),
    (2, 130, 768, 3072, 130, 70, torch.bfloat16), (2, 64, 200, 64, 64, 64, torch.float32), (2, 1, 64, 64, 5, 4, torch.bfloat16)])
def test_factmask_parity(G, W, oracle_mod, B, T, d_in, d_out, kin, kout, dtype):
    cfg = W.FactGrassWorkload("t", (W.LinearLayer("l", d_in, d_out),), B=B, T=T, kin=kin, kout=kout, k=1, data_seed=7)
    A, Gt = W.layer_io(cfg, 0, device="cuda", dtype=dtype)
    mi = oracle_mod.random_mask(d_in, kin, 1)
    mo = oracle_mod.random_mask(d_out, kout, 2)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = G.factmask_compress(A, Gt, G.mask_to_device(mi), G.mask_to_device(mo), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    f32 = dtype == torch.float32
    ref, absum = oracle_mod.factmask(W.bits_of(A), W.bits_of(Gt), mi, mo, dtype="f32" if f32 else "bf16")
    check_close(out.cpu().numpy(), ref, absum, 1e-4 if f32 else 2e-2, T + 64, eps=2.0 ** -23, what="factmask")


def test_factmask_grouped(G, W, oracle_mod):
    B, T = 2, 90
    specs = [(96, 160, 24, 40), (768, 768, 64, 64), (256, 512, 100, 70)]
    layers, keep, off = [], [], 0
    for n, (d_in, d_out, kin, kout) in enumerate(specs):
        cfg = W.FactGrassWorkload("t", (W.LinearLayer("l", d_in, d_out),), B=B, T=T, kin=kin, kout=kout, k=1, data_seed=30 + n)
        A, Gt = W.layer_io(cfg, 0, device="cuda")
        mi = oracle_mod.random_mask(d_in, kin, n)
        mo = oracle_mod.random_mask(d_out, kout, n + 9)
        layers.append(dict(A=A, G=Gt, mask_in=G.mask_to_device(mi), mask_out=G.mask_to_device(mo), k=1, s=1, seed=0,
                           out_offset=off))
        keep.append((off, kin * kout, mi, mo, A, Gt))
        off += kin * kout + 3
    out = torch.full((B, off), 5.0, device="cuda")
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(len(layers)), dtype=torch.uint8, device="cuda")
    G.factmask_compress_grouped(G.GroupedLayers(layers), out, ws)
    host = out.cpu().numpy()
    for (o, kp, mi, mo, A, Gt) in keep:
        ref, absum = oracle_mod.factmask(W.bits_of(A), W.bits_of(Gt), mi, mo)
        check_close(host[:, o:o + kp], ref, absum, 2e-2, T + 64, eps=2.0 ** -23, what=f"factmask grouped off={o}")
        assert np.all(host[:, o + kp:o + kp + 3] == 5.0)
