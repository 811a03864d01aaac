"""GPU parity of the bf16 cache path: grass_to_bf16 (bit-exact round to nearest even) and grass_score_bf16."""
import numpy as np
import pytest
import torch

from parity import check_close

pytestmark = pytest.mark.gpu

EPS_TC = 2.0 ** -23


@pytest.fixture(scope="module")
def G():
    import paper_2505_18976_b200 as g
    g.lib()
    return g


def _rne_bf16_bits(x: np.ndarray) -> np.ndarray:
    """fp32 -> bf16 bit patterns, round to nearest even, written out on the integer representation."""
    u = x.view(np.uint32).astype(np.uint64)
    nan = np.isnan(x)
    r = (u + 0x7FFF + ((u >> 16) & 1)) >> 16
    r = r.astype(np.uint16)
    r[nan] = ((u[nan] >> 16) | 0x40).astype(np.uint16)
    return r


def test_to_bf16_is_round_to_nearest_even(G):
    g = torch.Generator(device="cuda")
    g.manual_seed(4)
    x = torch.randn((37, 1_001), generator=g, device="cuda") * 10.0 ** torch.randint(-20, 20, (37, 1), device="cuda", generator=g)
    x[0, :6] = torch.tensor([0.0, -0.0, float("inf"), -float("inf"), 1.00390625, 1.01171875])   # two exact ties
    wide = torch.zeros((37, 1_008), device="cuda")
    wide[:, :1_001] = x
    out = G.grass_to_bf16(wide[:, :1_001])
    bits = out.view(torch.uint16).cpu().numpy()
    assert np.array_equal(bits, _rne_bf16_bits(np.ascontiguousarray(x.cpu().numpy())))


@pytest.mark.parametrize("N,M,D", [(300, 70, 264), (128, 128, 64), (1, 1, 8), (513, 256, 4096), (5, 3, 16),
                                   (257, 513, 104), (640, 40, 8), (2048, 256, 4096), (200, 100, 20_000)])
@pytest.mark.parametrize("solo", [1, 0])
def test_score_bf16_parity(G, oracle_mod, tune, N, M, D, solo):
    """Both kernels: one thread block per tile (taken for M <= 256) and thread-block pairs (any M)."""
    tune(score_bf16_solo=solo)
    g = torch.Generator(device="cuda")
    g.manual_seed(N + D)
    pad = 8 * (N % 3)
    trw = torch.randn((N, D + pad), generator=g, device="cuda").to(torch.bfloat16)
    tew = torch.randn((M, D + pad), generator=g, device="cuda").to(torch.bfloat16)
    tr, te = trw[:, :D], tew[:, :D]
    buf = torch.full((N, M + 3), 9.0, device="cuda")
    sc = G.grass_score_bf16(tr, te, out=buf[:, :M])
    ref, absum = oracle_mod.score(np.ascontiguousarray(tr.float().cpu().numpy()), np.ascontiguousarray(te.float().cpu().numpy()))
    check_close(sc.cpu().numpy(), ref, absum, 1e-4, D + 72, eps=EPS_TC, what=f"bf16 score {N}x{M}x{D}")
    assert torch.all(buf[:, M:] == 9.0)


def test_score_bf16_forced_splits_and_unsupported_strides(G, oracle_mod, tune):
    g = torch.Generator(device="cuda")
    g.manual_seed(3)
    tr = torch.randn((260, 1_000), generator=g, device="cuda").to(torch.bfloat16)
    te = torch.randn((90, 1_000), generator=g, device="cuda").to(torch.bfloat16)
    ref, absum = oracle_mod.score(tr.float().cpu().numpy(), te.float().cpu().numpy())
    for splits, solo in ((1, 1), (3, 1), (32, 1), (1, 0), (3, 0), (32, 0)):
        tune(score_splits=splits, score_bf16_solo=solo)
        sc = G.grass_score_bf16(tr, te, out=torch.full((260, 90), -1.0, device="cuda"))
        check_close(sc.cpu().numpy(), ref, absum, 1e-4, 1_000 + 72, eps=EPS_TC, what=f"bf16 score, {splits} splits")
    tune(score_splits=None, score_bf16_solo=None)
    with pytest.raises(G.GrassError) as e:
        G.grass_score_bf16(tr[:, :996][:, 1:], te[:, :996][:, 1:])          # base not 16-byte aligned
    assert e.value.code == 3


def test_score_of_a_bf16_cache_tracks_the_fp32_scores(G):
    """End to end: compressed fp32 vectors -> bf16 cache -> scores; against the fp32 scores the error is the
    rounding of the cache (2^-9 per entry, averaging out over D)."""
    g = torch.Generator(device="cuda")
    g.manual_seed(8)
    tr = torch.randn((512, 4_096), generator=g, device="cuda")
    te = torch.randn((64, 4_096), generator=g, device="cuda")
    full = G.grass_score(tr, te)
    half = G.grass_score_bf16(G.grass_to_bf16(tr), G.grass_to_bf16(te))
    scale = tr.norm(dim=1)[:, None] * te.norm(dim=1)[None, :]
    assert float(((full - half).abs() / scale).max()) < 2.0 ** -9
