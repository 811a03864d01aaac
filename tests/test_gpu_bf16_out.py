"""Compressed rows written as bf16 by the compress calls themselves (grass_compress_out,
factgrass_compress_grouped_out): every output is the fp32 result rounded to nearest even once, at the final store.
Checked against the oracle's fp64 values (one bf16 rounding, 2^-9, on top of the fp32 tolerance) and against the fp32
call's output rounded by torch."""
import dataclasses

import numpy as np
import pytest
import torch

from parity import check_close, max_bin_load

pytestmark = pytest.mark.gpu

TOL_OUT = 2.0 ** -8          # one rounding to bf16 (2^-9) and the fp32 arithmetic before it
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


def _same_as_rounded_fp32(out16, out32):
    """bf16 output against the fp32 output rounded by torch: equal, except where the order of the fp32 additions
    moved a value across a rounding boundary (then one bf16 step apart)."""
    want = out32.to(torch.bfloat16)
    same = (out16 == want).float().mean().item()
    assert same >= 0.995, same
    step = (out16.float() - want.float()).abs()
    assert bool((step <= out32.abs() * 2.0 ** -7 + 1e-30).all())


@pytest.mark.parametrize("tuning", [dict(), dict(compress_jsplit=1), dict(compress_jsplit=4), dict(compress_jsplit=20, compress_cluster=0),
                                    dict(compress_rows=1)])
def test_grass_compress_bf16_out(G, W, oracle_mod, tune, tuning):
    n, p, kp, k, seed = 9, 40_000, 9_000, 1_000, 17
    g = W.dense_gradients(n, p, 0.8, "normal", 1.0, 5, device="cuda")
    idx = oracle_mod.random_mask(p, kp, 3)
    didx = G.mask_to_device(idx)
    tune(**tuning)
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    buf = torch.full((n, k + 8), 3.0, dtype=torch.bfloat16, device="cuda")
    out16 = G.grass_compress(g, didx, k, 1, seed, out=buf[:, :k], dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and out16.dtype == torch.bfloat16
    assert torch.all(buf[:, k:] == 3.0)                       # columns beyond k untouched
    ref, absum = oracle_mod.grass(W.bits_of(g), idx, k, 1, seed)
    ob, _ = oracle_mod.sjlt_table(k, 1, seed, kp)
    check_close(out16.float().cpu().numpy(), ref, absum, TOL_OUT, max_bin_load(ob, k) + 16, what=f"bf16 out {tuning}")
    _same_as_rounded_fp32(out16, G.grass_compress(g, didx, k, 1, seed))


def test_grass_compress_bf16_out_identity_mask_and_bf16_input(G, W, oracle_mod):
    g = W.dense_gradients(6, 33_000, 0.9, "normal", 1.0, 8, device="cuda", dtype=torch.bfloat16)
    out16 = G.grass_compress(g, None, 512, 2, 4, out_dtype=torch.bfloat16)
    ref, absum = oracle_mod.grass(W.bits_of(g), None, 512, 2, 4, dtype="bf16", p=33_000)
    check_close(out16.float().cpu().numpy(), ref, absum, TOL_OUT, 200, what="bf16 in, bf16 out, s = 2")


def test_grass_compress_bf16_out_needs_shared_memory_bins(G):
    g = torch.randn(2, 70_000, device="cuda")
    with pytest.raises(G.GrassError) as e:
        G.grass_compress(g, None, 60_000, 1, 0, out_dtype=torch.bfloat16)       # 240 KB of bins: global reductions
    assert e.value.code == 3
    out = torch.full((2, 16), 5.0, dtype=torch.bfloat16, device="cuda")
    idx = torch.empty(0, dtype=torch.int32, device="cuda")
    G.grass_compress(g, idx, 16, 1, 0, out=out)                                  # empty mask: a zeroed bf16 row
    assert torch.all(out == 0)


def _layers(G, W, oracle_mod, cfg, ids):
    layers, refs = [], []
    for n, l in enumerate(ids):
        lay = cfg.layers[l]
        A, Gt = W.layer_io(cfg, l, device="cuda")
        s_in, s_out = W.layer_mask_seeds(cfg, l)
        mi = oracle_mod.random_mask(lay.d_in, cfg.kin, s_in)
        mo = oracle_mod.random_mask(lay.d_out, cfg.kout, s_out)
        layers.append(dict(A=A, G=Gt, mask_in=G.mask_to_device(mi), mask_out=G.mask_to_device(mo), k=cfg.k, s=cfg.s,
                           seed=W.layer_hash_seed(cfg, l), out_offset=n * cfg.k))
        refs.append((n * cfg.k, mi, mo, W.layer_hash_seed(cfg, l), A, Gt))
    return layers, refs


def test_factgrass_grouped_bf16_out(G, W, oracle_mod, fg_path):
    """Both kernels: the cluster kernel, and the streaming kernel with one thread block per (layer, sample)."""
    cfg = dataclasses.replace(W.CONFIG4, B=3, T=200, layers=W.CONFIG4.layers[:4])
    layers, refs = _layers(G, W, oracle_mod, cfg, range(4))
    group = G.GroupedLayers(layers)
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(4), dtype=torch.uint8, device="cuda")
    buf = torch.full((cfg.B, 4 * cfg.k + 6), 2.0, dtype=torch.bfloat16, device="cuda")
    st = torch.zeros(1, dtype=torch.int32, device="cuda")
    out16 = G.factgrass_compress_grouped(group, buf[:, :4 * cfg.k], ws, dev_status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0
    assert torch.all(buf[:, 4 * cfg.k:] == 2.0)
    host = out16.float().cpu().numpy()
    for (o, mi, mo, seed, A, Gt) in refs:
        ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, cfg.k, cfg.s, seed)
        check_close(host[:, o:o + cfg.k], ref, absum, 2e-2, cfg.T + 64, eps=EPS_TC, what=f"grouped bf16 out, off={o}")
    out32 = torch.empty((cfg.B, 4 * cfg.k), device="cuda")
    G.factgrass_compress_grouped(group, out32, ws)
    _same_as_rounded_fp32(out16, out32)


def test_factgrass_bf16_out_shapes_the_streaming_kernel_cannot_own(G, W, oracle_mod, tune):
    """A 128 x 128 block spans four tiles of the streaming kernel: bf16 rows then need the cluster kernel; with it
    switched off the call is refused instead of rounding partial sums."""
    cfg = dataclasses.replace(W.CONFIG3, B=2, T=96)
    layers, refs = _layers(G, W, oracle_mod, cfg, [0])
    group = G.GroupedLayers(layers)
    ws = torch.empty(G.factgrass_grouped_workspace_bytes(1), dtype=torch.uint8, device="cuda")
    out16 = torch.empty((cfg.B, cfg.k), dtype=torch.bfloat16, device="cuda")
    G.factgrass_compress_grouped(group, out16, ws)
    (o, mi, mo, seed, A, Gt) = refs[0]
    ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, cfg.k, cfg.s, seed)
    check_close(out16.float().cpu().numpy(), ref, absum, 2e-2, cfg.T + 64, eps=EPS_TC, what="128 x 128 block, bf16 out")
    tune(factgrass_path=0)
    with pytest.raises(G.GrassError) as e:
        G.factgrass_compress_grouped(group, out16, ws)
    assert e.value.code == 3


def test_bf16_rows_feed_the_bf16_score(G, W, oracle_mod):
    g = W.dense_gradients(96, 20_000, 0.7, "normal", 1.0, 2, device="cuda")
    idx = G.mask_to_device(oracle_mod.random_mask(20_000, 4_000, 0))
    c16 = G.grass_compress(g, idx, 512, 1, 9, out_dtype=torch.bfloat16)
    sc = G.grass_score_bf16(c16[:64], c16[64:])
    ref, absum = oracle_mod.score(c16[:64].float().cpu().numpy(), c16[64:].float().cpu().numpy())
    check_close(sc.cpu().numpy(), ref, absum, 1e-4, 512 + 72, eps=EPS_TC, what="score of bf16 rows")
