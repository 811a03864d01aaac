"""The workspace-free grouped entry point (for callers that cannot allocate device memory, such as a
hook running while the framework's pool holds all of HBM) must give what the ordinary grouped call
gives.  Collected last on purpose: a run that stops at the first failure has then already run every
other test.  Two calls in a row check that the shared descriptor table is rewritten per call."""
import dataclasses

import numpy as np
import pytest
import torch

from parity import check_close

pytestmark = pytest.mark.gpu


def _layers(G, W, oracle, cfg, ids):
    layers, extra = [], []
    for n, l in enumerate(ids):
        lay = cfg.layers[l]
        A, Gt = W.layer_io(cfg, l, device="cuda")
        s_in, s_out = W.layer_mask_seeds(cfg, l)
        mi = oracle.random_mask(lay.d_in, cfg.kin, s_in)
        mo = oracle.random_mask(lay.d_out, cfg.kout, s_out)
        seed = W.layer_hash_seed(cfg, l)
        layers.append(dict(A=A, G=Gt, mask_in=G.mask_to_device(mi), mask_out=G.mask_to_device(mo), k=cfg.k, s=cfg.s,
                           seed=seed, out_offset=n * cfg.k))
        extra.append((A, Gt, mi, mo, seed))
    return layers, extra


def test_static_table_entry_matches_workspace_entry(oracle_mod):
    import paper_2505_18976_b200 as G
    from paper_2505_18976_b200 import workloads as W
    assert G.FACTGRASS_STATIC_MAX_LAYERS == 256
    cfg = dataclasses.replace(W.CONFIG4, B=3, T=160, layers=W.CONFIG4.layers[:8])
    for call, ids in enumerate(([0, 1, 2, 3, 4], [7, 6, 5])):        # second call: other layers, fewer of them
        layers, extra = _layers(G, W, oracle_mod, cfg, ids)
        group = G.GroupedLayers(layers)
        width = cfg.k * len(ids)
        want = torch.empty(cfg.B, width, device="cuda")
        ws = torch.empty(G.factgrass_grouped_workspace_bytes(len(ids)), dtype=torch.uint8, device="cuda")
        G.factgrass_compress_grouped(group, want, ws)
        got = torch.full((cfg.B, width), 9.0, device="cuda")
        st = torch.zeros(1, dtype=torch.int32, device="cuda")
        G.factgrass_compress_grouped_static(group, got, dev_status=st)
        torch.cuda.synchronize()
        assert int(st.item()) == 0
        got_h, want_h = got.cpu().numpy(), want.cpu().numpy()
        for n, (A, Gt, mi, mo, seed) in enumerate(extra):
            ref, absum = oracle_mod.factgrass(W.bits_of(A), W.bits_of(Gt), mi, mo, cfg.k, cfg.s, seed)
            sl = slice(n * cfg.k, (n + 1) * cfg.k)
            # against the existing entry point, within the tolerance of the parity tests (the two runs may
            # differ in the order of their float additions)
            check_close(got_h[:, sl], want_h[:, sl].astype(np.float64), absum, 2e-2, cfg.T + 64, eps=2.0 ** -23,
                        what=f"static vs workspace, call {call}, layer {n}")
            check_close(got_h[:, sl], ref, absum, 2e-2, cfg.T + 64, eps=2.0 ** -23, what=f"static vs oracle, call {call}")


def test_static_table_entry_rejects_too_many_layers():
    import paper_2505_18976_b200 as G
    L = G.lib()
    arr = (G.FactgrassLayer * 257)()
    out = torch.zeros(1, 8, device="cuda")
    code = L.factgrass_compress_grouped_static(arr, 257, 1, 1, 8, out.data_ptr(), 8, None, None)
    assert code == 3                                                  # GRASS_ERR_UNSUPPORTED, nothing enqueued
    torch.cuda.synchronize()
    assert torch.all(out == 0)
