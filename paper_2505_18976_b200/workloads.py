"""Seeded synthetic workloads: shapes, value distributions and sparsity of the
five benchmark configurations, plus scaled-down variants for parity tests.

This module only *describes* and *draws* inputs (with ``torch.Generator``); it
holds none of the compression arithmetic (no hashing, no mask sampling, no
projection).  Both the CUDA path and the CPU oracle are fed the bytes drawn
here, so neither depends on the other for its inputs.

The tensors stand in for what the paper compresses: dense-but-sparse per-sample
gradients of MLP/ResNet-sized models (GraSS, Section 3.3.1) and the per-token
layer inputs / pre-activation gradients of GPT-2-small- and Llama-3-8B-shaped
linear layers (FactGraSS, Section 3.3.2; model sizes from the paper's Table 3).
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Tuple

import torch


# --------------------------------------------------------------------------- configs

@dataclass(frozen=True)
class GrassWorkload:
    """Dense per-sample gradients -> Mask_k' -> SJLT_k."""
    name: str
    n: int                # samples in the whole job
    batch: int            # samples per grass_compress call
    p: int                # gradient length
    kprime: int           # masked length k'
    k: int                # output length
    s: int = 1
    zero_prob: float = 0.0
    dist: str = "normal"  # "normal" | "student_t3"
    scale: float = 1.0
    dtype: str = "f32"
    data_seed: int = 0
    mask_seed: int = 0
    hash_seed: int = 0


@dataclass(frozen=True)
class LinearLayer:
    name: str
    d_in: int
    d_out: int


@dataclass(frozen=True)
class FactGrassWorkload:
    """Per-token (A, G) of linear layers -> factor masks -> Kronecker sum -> SJLT_k."""
    name: str
    layers: Tuple[LinearLayer, ...]
    B: int
    T: int
    kin: int
    kout: int
    k: int                 # output length per layer
    s: int = 1
    a_dist: str = "normal"
    a_scale: float = 1.0
    g_dist: str = "normal"  # "normal" | "laplace"
    g_scale: float = 1e-3
    pad_frac: float = 0.0   # trailing padding: pad_b ~ U{0..floor(2*pad_frac*T)}, G rows zeroed
    data_seed: int = 0
    mask_seed: int = 0
    hash_seed: int = 0
    # score step (config 5): compressed train vs test vectors
    score_n_train: int = 0
    score_n_test: int = 0

    @property
    def out_dim(self) -> int:
        return self.k * len(self.layers)


def _gpt2_small_layers(blocks: int = 12) -> Tuple[LinearLayer, ...]:
    out = []
    for b in range(blocks):
        out += [LinearLayer(f"h{b}.c_attn", 768, 2304), LinearLayer(f"h{b}.attn_c_proj", 768, 768),
                LinearLayer(f"h{b}.c_fc", 768, 3072), LinearLayer(f"h{b}.mlp_c_proj", 3072, 768)]
    return tuple(out)


def _llama3_8b_layers(blocks: int = 32) -> Tuple[LinearLayer, ...]:
    out = []
    for b in range(blocks):
        out += [LinearLayer(f"l{b}.q", 4096, 4096), LinearLayer(f"l{b}.k", 4096, 1024),
                LinearLayer(f"l{b}.v", 4096, 1024), LinearLayer(f"l{b}.o", 4096, 4096),
                LinearLayer(f"l{b}.gate", 4096, 14336), LinearLayer(f"l{b}.up", 4096, 14336),
                LinearLayer(f"l{b}.down", 14336, 4096)]
    return tuple(out)


CONFIG1 = GrassWorkload("c1_grass_p64k", n=256, batch=256, p=65_536, kprime=8_192, k=2_048,
                        zero_prob=0.9, dist="normal", scale=1.0,
                        data_seed=1001, mask_seed=0, hash_seed=0x5EED + 1)
CONFIG2 = GrassWorkload("c2_grass_p4m", n=4_096, batch=512, p=4_194_304, kprime=65_536, k=4_096,
                        zero_prob=0.7, dist="student_t3", scale=1e-2,
                        data_seed=1002, mask_seed=0, hash_seed=0x5EED + 2)
CONFIG3 = FactGrassWorkload("c3_factgrass_1layer", (LinearLayer("fc", 768, 3072),), B=32, T=512,
                            kin=128, kout=128, k=4_096, g_dist="normal", g_scale=1e-3,
                            pad_frac=0.05, data_seed=1003, mask_seed=3, hash_seed=0x5EED + 3)
CONFIG4 = FactGrassWorkload("c4_factgrass_gpt2s", _gpt2_small_layers(), B=16, T=1_024,
                            kin=64, kout=64, k=1_024, g_dist="laplace", g_scale=1e-3,
                            data_seed=1004, mask_seed=4, hash_seed=0x5EED + 4)
CONFIG5 = FactGrassWorkload("c5_factgrass_llama3_8b", _llama3_8b_layers(), B=4, T=2_048,
                            kin=64, kout=64, k=4_096, g_dist="normal", g_scale=1e-4,
                            data_seed=1005, mask_seed=5, hash_seed=0x5EED + 5,
                            score_n_train=16_384, score_n_test=256)

CONFIGS = {1: CONFIG1, 2: CONFIG2, 3: CONFIG3, 4: CONFIG4, 5: CONFIG5}


def scaled_down(cfg, **over):
    """A smaller workload with the same structure (for oracle-speed parity tests)."""
    return replace(cfg, **over)


# per-layer seeds of a FactGraSS workload: plain offsets, the hash does the mixing
def layer_hash_seed(cfg: FactGrassWorkload, l: int) -> int:
    return cfg.hash_seed + 7919 * l


def layer_mask_seeds(cfg: FactGrassWorkload, l: int) -> Tuple[int, int]:
    return cfg.mask_seed + 104_729 * (2 * l + 1), cfg.mask_seed + 104_729 * (2 * l + 2)


# --------------------------------------------------------------------------- draws

def _gen(device, seed: int) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(int(seed))
    return g


def dense_gradients(n: int, p: int, zero_prob: float, dist: str, scale: float, seed: int,
                    device="cpu", dtype=torch.float32, ld: int | None = None,
                    rows_per_chunk: int | None = None) -> torch.Tensor:
    """(n, ld) tensor (a view of width p is the data; columns >= p are NaN so a
    kernel that reads past p is caught).  Entries are exactly zero with
    probability ``zero_prob``; the others follow ``dist`` times ``scale``."""
    ld = p if ld is None else ld
    out = torch.empty((n, ld), dtype=dtype, device=device)
    if ld > p:
        out[:, p:] = float("nan")
    g = _gen(device, seed)
    if rows_per_chunk is None:
        rows_per_chunk = max(1, (64 << 20) // max(p, 1))
    for r0 in range(0, n, rows_per_chunk):
        r1 = min(n, r0 + rows_per_chunk)
        shape = (r1 - r0, p)
        z = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
        if dist == "student_t3":
            chi = torch.zeros(shape, device=device, dtype=torch.float32)
            for _ in range(3):
                w = torch.randn(shape, generator=g, device=device, dtype=torch.float32)
                chi.addcmul_(w, w)
            z = z / torch.sqrt(chi / 3.0)
        elif dist != "normal":
            raise ValueError(dist)
        z *= scale
        if zero_prob > 0:
            keep = torch.rand(shape, generator=g, device=device) >= zero_prob
            z = z * keep
        out[r0:r1, :p] = z.to(dtype)
    return out


def _draw(shape, dist: str, scale: float, g: torch.Generator, device) -> torch.Tensor:
    if dist == "normal":
        return torch.randn(shape, generator=g, device=device, dtype=torch.float32) * scale
    if dist == "laplace":
        u = torch.rand(shape, generator=g, device=device, dtype=torch.float32) - 0.5
        return -scale * torch.sign(u) * torch.log1p(-2.0 * u.abs().clamp(max=0.4999999))
    raise ValueError(dist)


def layer_io(cfg: FactGrassWorkload, l: int, device="cpu", dtype=torch.bfloat16):
    """(A, G) of layer ``l``: A (B,T,d_in), G (B,T,d_out), token-major contiguous."""
    lay = cfg.layers[l]
    g = _gen(device, cfg.data_seed + 1_000_003 * l)
    A = _draw((cfg.B, cfg.T, lay.d_in), cfg.a_dist, cfg.a_scale, g, device).to(dtype)
    G = _draw((cfg.B, cfg.T, lay.d_out), cfg.g_dist, cfg.g_scale, g, device).to(dtype)
    if cfg.pad_frac > 0:
        hi = int(2 * cfg.pad_frac * cfg.T)
        pads = torch.randint(0, hi + 1, (cfg.B,), generator=_gen("cpu", cfg.data_seed + 17 + l))
        for b in range(cfg.B):
            if int(pads[b]) > 0:
                G[b, cfg.T - int(pads[b]):, :] = 0
    return A, G


def score_vectors(n_train: int, n_test: int, D: int, seed: int, device="cpu"):
    """Stand-ins for compressed train / test gradients (fp32, N(0,1))."""
    g = _gen(device, seed)
    train = torch.randn((n_train, D), generator=g, device=device, dtype=torch.float32)
    test = torch.randn((n_test, D), generator=g, device=device, dtype=torch.float32)
    return train, test


# --------------------------------------------------------------------------- bytes

def unique_sectors(idx, elem_bytes: int, sector_bytes: int = 32) -> int:
    """Distinct ``sector_bytes``-sized sectors of one row that the mask touches."""
    per = sector_bytes // elem_bytes
    t = torch.as_tensor(idx.astype("int64") if hasattr(idx, "astype") else idx, dtype=torch.int64)
    return int(torch.unique(t // per).numel())


def bits_of(t: torch.Tensor):
    """numpy view of a CPU tensor's storage: float32 as is, bfloat16 as uint16."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.uint16).numpy()
    return t.numpy()
