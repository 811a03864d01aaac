"""GPU parity of the sequence-length-aware FactGraSS calls against the CPU oracle."""
import dataclasses

import numpy as np
import pytest
import torch

from parity import check_close, max_bin_load

pytestmark = pytest.mark.gpu

TOL_BF16, EPS_TC = 2e-2, 2.0 ** -23


@pytest.fixture(scope="module")
def G():
    import paper_2505_18976_b200 as g
    g.lib()
    return g


@pytest.fixture(scope="module")
def W():
    from paper_2505_18976_b200 import workloads
    return workloads


def _layer(G, W, oracle_mod, B, T, d_in, d_out, kin, kout, seed):
    cfg = W.FactGrassWorkload("t", (W.LinearLayer("l", d_in, d_out),), B=B, T=T, kin=kin, kout=kout, k=1, data_seed=seed)
    A, Gt = W.layer_io(cfg, 0, device="cuda")
    mi = oracle_mod.random_mask(d_in, kin, seed + 1)
    mo = oracle_mod.random_mask(d_out, kout, seed + 2)
    return A, Gt, mi, mo


def _i64(x):
    return torch.tensor(np.asarray(x), dtype=torch.int64, device="cuda")


def _i32(x):
    return torch.tensor(np.asarray(x), dtype=torch.int32, device="cuda")


@pytest.mark.parametrize("B,T,d_in,d_out,kin,kout,k,lens", [
    (5, 200, 96, 160, 24, 40, 97, [200, 0, 1, 77, 199]),
    (4, 300, 768, 3072, 128, 128, 4096, [300, 33, 256, 64]),          # config 3 tile shape, several chunks
    (3, 64, 200, 64, 64, 64, 1024, [5, 64, 31]),
])
def test_padded_batch_with_lengths(G, W, oracle_mod, B, T, d_in, d_out, kin, kout, k, lens, fg_path):
    A, Gt, mi, mo = _layer(G, W, oracle_mod, B, T, d_in, d_out, kin, kout, 40)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = G.factgrass_compress_varlen(A, Gt, G.mask_to_device(mi), G.mask_to_device(mo), k, 1, 123, B, T,
                                      tok_count=_i32(lens), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    ref, absum = oracle_mod.factgrass_varlen(W.bits_of(A).reshape(B * T, d_in), W.bits_of(Gt).reshape(B * T, d_out),
                                             mi, mo, k, 1, 123, np.arange(B) * T, lens)
    ob, _ = oracle_mod.sjlt_table(k, 1, 123, kin * kout)
    check_close(out.cpu().numpy(), ref, absum, TOL_BF16, T + max_bin_load(ob, k) + 64, eps=EPS_TC, what="padded varlen")
    for b, n in enumerate(lens):
        if n == 0:
            assert torch.all(out[b] == 0)


def test_packed_batch_grouped(G, W, oracle_mod, fg_path):
    """Three layers over one packed token stream (no padding rows), samples listed out of order."""
    lens = np.array([130, 7, 64, 0, 95], dtype=np.int32)
    begin = np.concatenate([[0], np.cumsum(lens)[:-1]]).astype(np.int64)
    rows, B, T_max = int(lens.sum()), len(lens), 130
    order = np.array([2, 0, 4, 1, 3])
    specs = [(96, 160, 24, 40, 97, 1), (768, 768, 64, 64, 1024, 1), (256, 512, 100, 70, 300, 2)]
    layers, keep, off = [], [], 0
    for n, (d_in, d_out, kin, kout, k, s) in enumerate(specs):
        A, Gt, mi, mo = _layer(G, W, oracle_mod, 1, rows, d_in, d_out, kin, kout, 60 + n)
        A, Gt = A[0].contiguous(), Gt[0].contiguous()
        layers.append(dict(A=A, G=Gt, mask_in=G.mask_to_device(mi), mask_out=G.mask_to_device(mo), k=k, s=s,
                           seed=9 + n, out_offset=off))
        keep.append((off, k, s, 9 + n, mi, mo, A, Gt, kin, kout))
        off += k
    out = torch.full((B, off), float("nan"), device="cuda")
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(len(layers)), dtype=torch.uint8, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    G.factgrass_compress_grouped_varlen(G.GroupedLayers(layers), out, ws, B, T_max, tok_begin=_i64(begin[order]),
                                        tok_count=_i32(lens[order]), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    host = out.cpu().numpy()
    for (o, k, s, seed, mi, mo, A, Gt, kin, kout) in keep:
        ref, absum = oracle_mod.factgrass_varlen(W.bits_of(A), W.bits_of(Gt), mi, mo, k, s, seed, begin[order], lens[order])
        ob, _ = oracle_mod.sjlt_table(k, s, seed, kin * kout)
        check_close(host[:, o:o + k], ref, absum, TOL_BF16, T_max + max_bin_load(ob, k) + 64, eps=EPS_TC,
                    what=f"packed grouped off={o}")


def test_null_arrays_equal_the_plain_call(G, W, oracle_mod, fg_path):
    A, Gt, mi, mo = _layer(G, W, oracle_mod, 3, 100, 96, 160, 24, 40, 70)
    dmi, dmo = G.mask_to_device(mi), G.mask_to_device(mo)
    a = G.factgrass_compress(A, Gt, dmi, dmo, 97, 1, 5)
    b = G.factgrass_compress_varlen(A, Gt, dmi, dmo, 97, 1, 5, 3, 100)
    assert float((a - b).abs().max()) <= 1e-5 * float(a.abs().max())


def test_lengths_out_of_range_are_clamped_and_flagged(G, W, oracle_mod, fg_path):
    B, T = 3, 50
    A, Gt, mi, mo = _layer(G, W, oracle_mod, B, T, 96, 160, 24, 40, 80)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out = G.factgrass_compress_varlen(A, Gt, G.mask_to_device(mi), G.mask_to_device(mo), 97, 1, 5, B, T,
                                      tok_count=_i32([60, -4, 20]), dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == G.binding.DEV_BAD_LENGTH
    ref, absum = oracle_mod.factgrass_varlen(W.bits_of(A).reshape(B * T, 96), W.bits_of(Gt).reshape(B * T, 160), mi, mo,
                                             97, 1, 5, np.arange(B) * T, [50, 0, 20])
    check_close(out.cpu().numpy(), ref, absum, TOL_BF16, T + 64, eps=EPS_TC, what="clamped lengths")


def test_config3_padding_skipped(G, W, oracle_mod, fg_path):
    """Config 3's trailing padding (zero output-gradient rows): passing the lengths gives the same
    compressed gradients as reading the zero rows."""
    c = dataclasses.replace(W.CONFIG3, B=8)
    A, Gt = W.layer_io(c, 0, device="cuda")
    lens = (Gt.abs().amax(dim=2) > 0).int().sum(dim=1).int()          # trailing all-zero rows are padding
    assert int(lens.min()) < c.T
    s_in, s_out = W.layer_mask_seeds(c, 0)
    mi = oracle_mod.random_mask(768, c.kin, s_in)
    mo = oracle_mod.random_mask(3072, c.kout, s_out)
    dmi, dmo = G.mask_to_device(mi), G.mask_to_device(mo)
    seed = W.layer_hash_seed(c, 0)
    full = G.factgrass_compress(A, Gt, dmi, dmo, c.k, 1, seed)
    short = G.factgrass_compress_varlen(A, Gt, dmi, dmo, c.k, 1, seed, c.B, c.T, tok_count=lens.contiguous())
    ref, absum = oracle_mod.factgrass_varlen(W.bits_of(A).reshape(c.B * c.T, 768), W.bits_of(Gt).reshape(c.B * c.T, 3072),
                                             mi, mo, c.k, 1, seed, np.arange(c.B) * c.T, lens.cpu().numpy())
    check_close(short.cpu().numpy(), ref, absum, TOL_BF16, c.T + 64, eps=EPS_TC, what="config 3 lengths")
    check_close(full.cpu().numpy(), ref, absum, TOL_BF16, c.T + 64, eps=EPS_TC, what="config 3 padded")
