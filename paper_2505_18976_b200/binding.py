"""Thin ctypes binding of ``libgrass_b200.so`` (declared in ``include/grass.h``).

Argument marshalling only: every step of the compression path runs in the CUDA
kernels behind the C ABI.  Functions take torch CUDA tensors (or raw integer
device pointers) and enqueue on torch's current stream.  There is no CPU
fallback: if the shared library is missing, loading raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

HERE = os.path.dirname(os.path.abspath(__file__))
SO_PATH = os.environ.get("GRASS_B200_LIB") or os.path.join(HERE, "libgrass_b200.so")

GRASS_OK = 0
STATUS = {0: "GRASS_OK", 1: "GRASS_ERR_INVALID_ARG", 2: "GRASS_ERR_BAD_MASK", 3: "GRASS_ERR_UNSUPPORTED",
          4: "GRASS_ERR_CUDA", 5: "GRASS_ERR_TIMEOUT"}
F32, BF16 = 0, 1
DEV_BAD_INDEX, DEV_TIMEOUT, DEV_BAD_LENGTH, DEV_NOT_PD = 1, 2, 4, 8

EXPORTS = ("grass_compress", "factgrass_compress", "factgrass_compress_grouped",
           "factgrass_compress_varlen", "factgrass_compress_grouped_varlen",
           "grass_fim", "grass_fim_factor", "grass_fim_apply", "grass_mask", "factmask_compress",
           "factmask_compress_grouped",
           "factgrass_grouped_workspace_bytes", "factgrass_compress_grouped_static", "grass_score", "grass_sjlt_table", "grass_validate_mask",
           "grass_random_mask_host", "grass_status_string", "grass_to_bf16", "grass_score_bf16", "grass_set_tuning",
           "grass_compress_out", "factgrass_compress_grouped_out")

# grass_tuning_key in include/grass.h
TUNE = {"compress_samples": 0, "compress_jsplit": 1, "compress_cluster": 2, "compress_dense": 3,
        "factgrass_tile": 4, "factgrass_chunk": 5, "factgrass_carveout": 6, "score_ffma": 7, "score_splits": 8,
        "split_products": 9, "factgrass_path": 10, "compress_rows": 11, "compress_loads": 12,
        "compress_threads": 13, "compress_idx_smem": 14, "score_bf16_solo": 15}


class GrassError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {STATUS.get(code, code)} ({lib().grass_status_string(code).decode()})")


class SjltSpec(ctypes.Structure):
    _fields_ = [("k", ctypes.c_uint32), ("s", ctypes.c_uint32), ("seed", ctypes.c_uint64)]


class FactgrassLayer(ctypes.Structure):
    _fields_ = [("A", ctypes.c_void_p), ("G", ctypes.c_void_p), ("mask_in", ctypes.c_void_p),
                ("mask_out", ctypes.c_void_p), ("d_in", ctypes.c_int32), ("d_out", ctypes.c_int32),
                ("kin", ctypes.c_int32), ("kout", ctypes.c_int32), ("spec", SjltSpec),
                ("out_offset", ctypes.c_int64)]


_lib = None


def lib() -> ctypes.CDLL:
    """Load the CUDA library; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(SO_PATH):
            raise ImportError(f"{SO_PATH} is missing: build it with `python -m paper_2505_18976_b200.build` "
                              "(there is no CPU fallback)")
        L = ctypes.CDLL(SO_PATH)
        i64, i32, vp, st = ctypes.c_int64, ctypes.c_int32, ctypes.c_void_p, ctypes.c_int
        sp = ctypes.POINTER(SjltSpec)
        L.grass_compress.restype = st
        L.grass_compress.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, i64, sp, vp, i64, vp, vp]
        L.grass_compress_out.restype = st
        L.grass_compress_out.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, i64, sp, vp, ctypes.c_int, i64, vp, vp]
        L.factgrass_compress_grouped_out.restype = st
        L.factgrass_compress_grouped_out.argtypes = [ctypes.POINTER(FactgrassLayer), i32, ctypes.c_int, i32, i32, vp,
                                                     ctypes.c_int, i64, vp, ctypes.c_size_t, vp, vp]
        L.factgrass_compress.restype = st
        L.factgrass_compress.argtypes = [vp, vp, ctypes.c_int, i32, i32, i32, i32, vp, i32, vp, i32, sp, vp, i64, vp, vp]
        L.factgrass_compress_grouped.restype = st
        L.factgrass_compress_grouped.argtypes = [ctypes.POINTER(FactgrassLayer), i32, ctypes.c_int, i32, i32, vp, i64,
                                                 vp, ctypes.c_size_t, vp, vp]
        L.factgrass_compress_varlen.restype = st
        L.factgrass_compress_varlen.argtypes = [vp, vp, ctypes.c_int, i32, i32, vp, vp, i32, i32, vp, i32, vp, i32, sp,
                                                vp, i64, vp, vp]
        L.factgrass_compress_grouped_varlen.restype = st
        L.factgrass_compress_grouped_varlen.argtypes = [ctypes.POINTER(FactgrassLayer), i32, ctypes.c_int, i32, i32,
                                                        vp, vp, vp, i64, vp, ctypes.c_size_t, vp, vp]
        L.factgrass_grouped_workspace_bytes.restype = ctypes.c_size_t
        L.factgrass_grouped_workspace_bytes.argtypes = [i32]
        L.factgrass_compress_grouped_static.restype = st
        L.factgrass_compress_grouped_static.argtypes = [ctypes.POINTER(FactgrassLayer), i32, ctypes.c_int, i32, i32, vp,
                                                        i64, vp, vp]
        L.grass_score.restype = st
        L.grass_score.argtypes = [vp, i64, i64, vp, i64, i64, i64, vp, i64, vp]
        L.grass_score_bf16.restype = st
        L.grass_score_bf16.argtypes = [vp, i64, i64, vp, i64, i64, i64, vp, i64, vp]
        L.grass_to_bf16.restype = st
        L.grass_to_bf16.argtypes = [vp, i64, i64, i64, vp, i64, vp]
        L.grass_mask.restype = st
        L.grass_mask.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, i64, vp, i64, vp, vp]
        L.factmask_compress.restype = st
        L.factmask_compress.argtypes = [vp, vp, ctypes.c_int, i32, i32, i32, i32, vp, i32, vp, i32, vp, i64, vp, vp]
        L.factmask_compress_grouped.restype = st
        L.factmask_compress_grouped.argtypes = [ctypes.POINTER(FactgrassLayer), i32, ctypes.c_int, i32, i32, vp, i64,
                                                vp, ctypes.c_size_t, vp, vp]
        L.grass_fim.restype = st
        L.grass_fim.argtypes = [vp, i64, i64, i64, vp, i64, vp]
        L.grass_fim_factor.restype = st
        L.grass_fim_factor.argtypes = [vp, i64, i64, ctypes.c_float, vp, vp]
        L.grass_fim_apply.restype = st
        L.grass_fim_apply.argtypes = [vp, i64, i64, vp, i64, i64, vp]
        L.grass_sjlt_table.restype = st
        L.grass_sjlt_table.argtypes = [sp, i64, vp, vp, vp]
        L.grass_validate_mask.restype = st
        L.grass_validate_mask.argtypes = [vp, i64, i64, vp]
        L.grass_random_mask_host.restype = st
        L.grass_random_mask_host.argtypes = [i64, i64, ctypes.c_uint64, vp]
        L.grass_set_tuning.restype = st
        L.grass_set_tuning.argtypes = [ctypes.c_int, i64]
        L.grass_status_string.restype = ctypes.c_char_p
        L.grass_status_string.argtypes = [st]
        _lib = L
    return _lib


def _check(code: int, where: str) -> None:
    if code != GRASS_OK:
        raise GrassError(code, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _ptr(t) -> Optional[int]:
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _dt(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return F32
    if t.dtype == torch.bfloat16:
        return BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _need_cuda(*ts) -> None:
    for t in ts:
        if t is not None and not isinstance(t, int) and not t.is_cuda:
            raise ValueError("device tensors required (the library has no CPU path)")


def _need_device_readable(*ts) -> None:
    """Inputs the kernels only gather from: device tensors, or page-locked host tensors (which the device
    addresses directly; the kernels then pull the masked elements across the bus)."""
    for t in ts:
        if t is not None and not (t.is_cuda or t.is_pinned()):
            raise ValueError("device or pinned host tensors required (the library has no CPU path)")


def _need_mask(*ms) -> None:
    """Index lists are read as uint32: a 4-byte integer dtype, contiguous."""
    for m in ms:
        if m is not None and not isinstance(m, int):
            if m.dtype not in (torch.int32, torch.uint32) or not m.is_contiguous() or m.dim() != 1:
                raise TypeError("mask index lists must be contiguous 1-D int32/uint32 tensors")


def grass_set_tuning(name: str, value: Optional[int]) -> None:
    """Force one launch-shape choice of the library (a test and measurement hook); None restores automatic."""
    _check(lib().grass_set_tuning(TUNE[name], -1 if value is None else int(value)), "grass_set_tuning")


class tuning:
    """Context manager: ``with tuning(factgrass_tile=128): ...`` forces the given choices and restores
    automatic ones on exit."""

    def __init__(self, **kw):
        self.kw = kw

    def __enter__(self):
        for k, v in self.kw.items():
            grass_set_tuning(k, v)
        return self

    def __exit__(self, *exc):
        for k in self.kw:
            grass_set_tuning(k, None)
        return False


def _compute_device(t: torch.Tensor) -> torch.device:
    return t.device if t.is_cuda else torch.device("cuda", torch.cuda.current_device())


def grass_compress(g: torch.Tensor, idx: Optional[torch.Tensor], k: int, s: int, seed: int,
                   out: Optional[torch.Tensor] = None, p: Optional[int] = None,
                   dev_status: Optional[torch.Tensor] = None, out_dtype: torch.dtype = torch.float32) -> torch.Tensor:
    """out[i] = SJLT_{k,s,seed}(g[i, idx]) for the rows of g (n x ld, fp32 or bf16).
    idx: uint32/int32 CUDA tensor of ascending coordinates, or None for the identity mask.
    g may be a pinned host tensor: the kernel then reads the masked elements in place, across the bus.
    The rows are written as fp32, or as bf16 (rounded once, at the final store) when `out` / `out_dtype` is bf16."""
    _need_device_readable(g)
    _need_cuda(idx, out, dev_status)
    _need_mask(idx)
    assert g.dim() == 2 and g.stride(1) == 1
    n, ld = g.shape[0], g.stride(0) if g.shape[0] > 1 else g.shape[1]
    p = g.shape[1] if p is None else p
    kprime = p if idx is None else idx.numel()
    if out is None:
        out = torch.empty((n, k), dtype=out_dtype, device=_compute_device(g))
    assert out.dtype in (torch.float32, torch.bfloat16) and out.stride(1) == 1
    spec = SjltSpec(k, s, seed & 0xFFFFFFFFFFFFFFFF)
    _check(lib().grass_compress_out(_ptr(g), _dt(g), n, p, ld, _ptr(idx), kprime, ctypes.byref(spec), _ptr(out),
                                    _dt(out), out.stride(0) if n > 1 else max(out.shape[1], k), _ptr(dev_status),
                                    _stream()), "grass_compress")
    return out


def factgrass_compress(A: torch.Tensor, G: torch.Tensor, mask_in: torch.Tensor, mask_out: torch.Tensor,
                       k: int, s: int, seed: int, out: Optional[torch.Tensor] = None,
                       dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """One linear layer: out[b] = SJLT(vec(sum_t A[b,t,mask_in] (x) G[b,t,mask_out]))."""
    _need_device_readable(A, G)
    _need_cuda(mask_in, mask_out, out, dev_status)
    _need_mask(mask_in, mask_out)
    assert A.is_contiguous() and G.is_contiguous() and A.dim() == 3 and G.dim() == 3
    B, T, d_in = A.shape
    d_out = G.shape[2]
    assert G.shape[:2] == (B, T) and A.dtype == G.dtype
    if out is None:
        out = torch.empty((B, k), dtype=torch.float32, device=_compute_device(A))
    spec = SjltSpec(k, s, seed & 0xFFFFFFFFFFFFFFFF)
    _check(lib().factgrass_compress(_ptr(A), _ptr(G), _dt(A), B, T, d_in, d_out, _ptr(mask_in), mask_in.numel(),
                                    _ptr(mask_out), mask_out.numel(), ctypes.byref(spec), _ptr(out),
                                    out.stride(0) if B > 1 else max(out.shape[1], k), _ptr(dev_status), _stream()),
           "factgrass_compress")
    return out


def _check_token_arrays(tok_begin, tok_count, B):
    _need_cuda(tok_begin, tok_count)
    if tok_begin is not None:
        assert tok_begin.dtype == torch.int64 and tok_begin.numel() == B and tok_begin.is_contiguous()
    if tok_count is not None:
        assert tok_count.dtype == torch.int32 and tok_count.numel() == B and tok_count.is_contiguous()


def factgrass_compress_varlen(A: torch.Tensor, G: torch.Tensor, mask_in: torch.Tensor, mask_out: torch.Tensor,
                              k: int, s: int, seed: int, B: int, T_max: int,
                              tok_begin: Optional[torch.Tensor] = None, tok_count: Optional[torch.Tensor] = None,
                              out: Optional[torch.Tensor] = None,
                              dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """One linear layer, samples with their own sequence lengths.  A, G: token-major (rows, d) matrices
    (or (B, T_max, d) for a padded batch); sample b owns rows tok_begin[b] .. + tok_count[b] (int64 /
    int32 CUDA tensors; None = b * T_max / T_max)."""
    _need_device_readable(A, G)
    _need_cuda(mask_in, mask_out, out, dev_status)
    _need_mask(mask_in, mask_out)
    assert A.is_contiguous() and G.is_contiguous() and A.dtype == G.dtype
    _check_token_arrays(tok_begin, tok_count, B)
    d_in, d_out = A.shape[-1], G.shape[-1]
    if tok_begin is None:
        assert A.numel() >= B * T_max * d_in and G.numel() >= B * T_max * d_out
    if out is None:
        out = torch.empty((B, k), dtype=torch.float32, device=_compute_device(A))
    spec = SjltSpec(k, s, seed & 0xFFFFFFFFFFFFFFFF)
    _check(lib().factgrass_compress_varlen(_ptr(A), _ptr(G), _dt(A), B, T_max, _ptr(tok_begin), _ptr(tok_count),
                                           d_in, d_out, _ptr(mask_in), mask_in.numel(), _ptr(mask_out),
                                           mask_out.numel(), ctypes.byref(spec), _ptr(out),
                                           out.stride(0) if B > 1 else max(out.shape[1], k), _ptr(dev_status),
                                           _stream()), "factgrass_compress_varlen")
    return out


class GroupedLayers:
    """Host-side descriptor table for factgrass_compress_grouped; keeps the tensors alive."""

    def __init__(self, layers: Sequence[dict]):
        """layers: dicts with A, G (CUDA tensors, or pinned host tensors read in place), mask_in, mask_out (CUDA
        tensors), k, s, seed, out_offset."""
        self.keep = list(layers)
        self.L = len(layers)
        self.array = (FactgrassLayer * max(self.L, 1))()
        for i, l in enumerate(layers):
            _need_device_readable(l["A"], l["G"])
            _need_cuda(l["mask_in"], l["mask_out"])
            _need_mask(l["mask_in"], l["mask_out"])
            A0, Al, Gl = layers[0]["A"], l["A"], l["G"]
            # every layer shares the token layout and dtype of the first; the kernels index with these
            if not (Al.is_contiguous() and Gl.is_contiguous()):
                raise ValueError(f"layer {i}: A and G must be contiguous")
            if Al.dim() != A0.dim() or Gl.dim() != A0.dim() or Al.shape[:-1] != A0.shape[:-1] or \
                    Gl.shape[:-1] != A0.shape[:-1]:
                raise ValueError(f"layer {i}: A and G must share the leading (sample, token) shape of layer 0")
            if Al.dtype != A0.dtype or Gl.dtype != A0.dtype:
                raise TypeError(f"layer {i}: A and G must have the dtype of layer 0")
            if l["out_offset"] < 0:
                raise ValueError(f"layer {i}: negative out_offset")
            e = self.array[i]
            e.A, e.G = l["A"].data_ptr(), l["G"].data_ptr()
            e.mask_in, e.mask_out = l["mask_in"].data_ptr(), l["mask_out"].data_ptr()
            e.d_in, e.d_out = l["A"].shape[-1], l["G"].shape[-1]
            e.kin, e.kout = l["mask_in"].numel(), l["mask_out"].numel()
            e.spec = SjltSpec(l["k"], l["s"], l["seed"] & 0xFFFFFFFFFFFFFFFF)
            e.out_offset = l["out_offset"]
        self.dtype = _dt(layers[0]["A"]) if layers else BF16
        self.B, self.T = (layers[0]["A"].shape[0], layers[0]["A"].shape[1]) if layers else (0, 0)


def factgrass_grouped_workspace_bytes(L: int) -> int:
    return int(lib().factgrass_grouped_workspace_bytes(L))


def factgrass_compress_grouped(group: GroupedLayers, out: torch.Tensor, workspace: torch.Tensor,
                               dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """All layers of ``group`` in one launch; layer l fills out[:, off_l : off_l + k_l].  `out` is fp32, or bf16
    (every output rounded once, at the final store; see factgrass_compress_grouped_out in include/grass.h)."""
    _need_cuda(out, workspace, dev_status)
    assert out.dtype in (torch.float32, torch.bfloat16) and out.stride(1) == 1
    _check(lib().factgrass_compress_grouped_out(group.array, group.L, group.dtype, group.B, group.T, _ptr(out),
                                                _dt(out), out.stride(0) if out.shape[0] > 1 else out.shape[1],
                                                _ptr(workspace), workspace.numel() * workspace.element_size(),
                                                _ptr(dev_status), _stream()), "factgrass_compress_grouped")
    return out


def factgrass_compress_grouped_varlen(group: GroupedLayers, out: torch.Tensor, workspace: torch.Tensor, B: int,
                                      T_max: int, tok_begin: Optional[torch.Tensor] = None,
                                      tok_count: Optional[torch.Tensor] = None,
                                      dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """All layers of ``group`` in one launch for a batch whose samples have their own lengths; the layers'
    A and G are token-major (rows, d) matrices that share one token layout (tok_begin, tok_count)."""
    _need_cuda(out, workspace, dev_status)
    _check_token_arrays(tok_begin, tok_count, B)
    assert out.dtype == torch.float32 and out.stride(1) == 1 and out.shape[0] == B
    _check(lib().factgrass_compress_grouped_varlen(group.array, group.L, group.dtype, B, T_max, _ptr(tok_begin),
                                                   _ptr(tok_count), _ptr(out),
                                                   out.stride(0) if out.shape[0] > 1 else out.shape[1],
                                                   _ptr(workspace), workspace.numel() * workspace.element_size(),
                                                   _ptr(dev_status), _stream()), "factgrass_compress_grouped_varlen")
    return out


FACTGRASS_STATIC_MAX_LAYERS = 256   # FACTGRASS_STATIC_MAX_LAYERS in include/grass.h


def factgrass_compress_grouped_static(group: GroupedLayers, out: torch.Tensor,
                                      dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Grouped FactGraSS for callers that cannot allocate a device workspace (for example a hook running
    while the framework's memory pool owns all of HBM): the descriptor table sits in a fixed array inside
    the library, at most FACTGRASS_STATIC_MAX_LAYERS layers per call.  Calls share that table, so keep
    them on one stream; the first call on a device should happen outside stream capture."""
    _need_cuda(out, dev_status)
    assert out.dtype == torch.float32 and out.stride(1) == 1
    _check(lib().factgrass_compress_grouped_static(group.array, group.L, group.dtype, group.B, group.T, _ptr(out),
                                                   out.stride(0) if out.shape[0] > 1 else out.shape[1],
                                                   _ptr(dev_status), _stream()), "factgrass_compress_grouped_static")
    return out


def grass_score(train: torch.Tensor, test: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """scores[i, m] = <train[i], test[m]> (fp32)."""
    _need_cuda(train, test, out)
    assert train.dtype == torch.float32 and test.dtype == torch.float32
    assert train.stride(1) == 1 and test.stride(1) == 1
    N, D = train.shape
    M = test.shape[0]
    assert test.shape[1] == D
    if out is None:
        out = torch.empty((N, M), dtype=torch.float32, device=train.device)
    _check(lib().grass_score(_ptr(train), N, train.stride(0) if N > 1 else D, _ptr(test), M,
                             test.stride(0) if M > 1 else D, D, _ptr(out), out.stride(0) if N > 1 else M,
                             _stream()), "grass_score")
    return out


def grass_to_bf16(x: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Compressed vectors as bf16 (round to nearest even), for a cache at half the size."""
    _need_cuda(x, out)
    assert x.dtype == torch.float32 and x.dim() == 2 and x.stride(1) == 1
    n, k = x.shape
    if out is None:
        out = torch.empty((n, k), dtype=torch.bfloat16, device=x.device)
    assert out.dtype == torch.bfloat16 and out.stride(1) == 1
    for r0 in range(0, n, 65_535):
        r1 = min(n, r0 + 65_535)
        _check(lib().grass_to_bf16(_ptr(x[r0:r1]), r1 - r0, k, x.stride(0) if n > 1 else k, _ptr(out[r0:r1]),
                                   out.stride(0) if n > 1 else k, _stream()), "grass_to_bf16")
    return out


def grass_score_bf16(train: torch.Tensor, test: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """scores[i, m] = <train[i], test[m]> for bf16 vectors (fp32 scores)."""
    _need_cuda(train, test, out)
    assert train.dtype == torch.bfloat16 and test.dtype == torch.bfloat16
    assert train.stride(1) == 1 and test.stride(1) == 1
    N, D = train.shape
    M = test.shape[0]
    assert test.shape[1] == D
    if out is None:
        out = torch.empty((N, M), dtype=torch.float32, device=train.device)
    _check(lib().grass_score_bf16(_ptr(train), N, train.stride(0) if N > 1 else D, _ptr(test), M,
                                  test.stride(0) if M > 1 else D, D, _ptr(out), out.stride(0) if N > 1 else M,
                                  _stream()), "grass_score_bf16")
    return out


def grass_mask(g: torch.Tensor, idx: torch.Tensor, out: Optional[torch.Tensor] = None, p: Optional[int] = None,
               dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Stand-alone Mask: out[i, j] = g[i, idx[j]] as fp32.  g may be a pinned host tensor (read in place)."""
    _need_device_readable(g)
    _need_cuda(idx, out, dev_status)
    _need_mask(idx)
    assert g.dim() == 2 and g.stride(1) == 1
    n, ld = g.shape[0], g.stride(0) if g.shape[0] > 1 else g.shape[1]
    p = g.shape[1] if p is None else p
    kp = idx.numel()
    if out is None:
        out = torch.empty((n, kp), dtype=torch.float32, device=_compute_device(g))
    _check(lib().grass_mask(_ptr(g), _dt(g), n, p, ld, _ptr(idx), kp, _ptr(out),
                            out.stride(0) if n > 1 else max(out.shape[1], kp), _ptr(dev_status), _stream()), "grass_mask")
    return out


def factmask_compress(A: torch.Tensor, G: torch.Tensor, mask_in: torch.Tensor, mask_out: torch.Tensor,
                      out: Optional[torch.Tensor] = None, dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Factorised Mask of one linear layer: out[b, a*kout + c] = sum_t A[b,t,mask_in[a]] G[b,t,mask_out[c]]."""
    _need_device_readable(A, G)
    _need_cuda(mask_in, mask_out, out, dev_status)
    _need_mask(mask_in, mask_out)
    assert A.is_contiguous() and G.is_contiguous() and A.dim() == 3 and G.dim() == 3 and A.dtype == G.dtype
    assert G.shape[:2] == A.shape[:2]
    B, T, d_in = A.shape
    d_out = G.shape[2]
    kin = d_in if mask_in is None else mask_in.numel()          # None = identity mask
    kout = d_out if mask_out is None else mask_out.numel()
    kp = kin * kout
    if out is None:
        out = torch.empty((B, kp), dtype=torch.float32, device=_compute_device(A))
    _check(lib().factmask_compress(_ptr(A), _ptr(G), _dt(A), B, T, d_in, d_out, _ptr(mask_in), kin,
                                   _ptr(mask_out), kout, _ptr(out),
                                   out.stride(0) if B > 1 else max(out.shape[1], kp), _ptr(dev_status), _stream()),
           "factmask_compress")
    return out


def factmask_compress_grouped(group: "GroupedLayers", out: torch.Tensor, workspace: torch.Tensor,
                              dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """Factorised Mask of all layers of ``group`` in one launch (the layers' k, s, seed are ignored)."""
    _need_cuda(out, workspace, dev_status)
    assert out.dtype == torch.float32 and out.stride(1) == 1
    _check(lib().factmask_compress_grouped(group.array, group.L, group.dtype, group.B, group.T, _ptr(out),
                                           out.stride(0) if out.shape[0] > 1 else out.shape[1], _ptr(workspace),
                                           workspace.numel() * workspace.element_size(), _ptr(dev_status),
                                           _stream()), "factmask_compress_grouped")
    return out


def grass_fim(X: torch.Tensor, out: Optional[torch.Tensor] = None) -> torch.Tensor:
    """F = X^T X / n for the n rows of X (fp32; a column slice of a wider matrix is fine)."""
    _need_cuda(X, out)
    assert X.dtype == torch.float32 and X.dim() == 2 and X.stride(1) == 1
    n, k = X.shape
    if out is None:
        out = torch.empty((k, k), dtype=torch.float32, device=X.device)
    assert out.dtype == torch.float32 and out.stride(1) == 1 and out.shape == (k, k)
    _check(lib().grass_fim(_ptr(X), n, k, X.stride(0) if n > 1 else max(k, X.stride(0)), _ptr(out),
                           out.stride(0) if k > 1 else max(k, 1), _stream()), "grass_fim")
    return out


def grass_fim_factor(F: torch.Tensor, lam: float, dev_status: Optional[torch.Tensor] = None) -> torch.Tensor:
    """In place: lower triangle of F <- Cholesky factor of F + lam * I."""
    _need_cuda(F, dev_status)
    assert F.dtype == torch.float32 and F.dim() == 2 and F.shape[0] == F.shape[1] and F.stride(1) == 1
    k = F.shape[0]
    _check(lib().grass_fim_factor(_ptr(F), k, F.stride(0) if k > 1 else 1, float(lam), _ptr(dev_status), _stream()),
           "grass_fim_factor")
    return F


def grass_fim_apply(L: torch.Tensor, Bm: torch.Tensor) -> torch.Tensor:
    """In place: every row b of Bm <- (L L^T)^-1 b, L from grass_fim_factor."""
    _need_cuda(L, Bm)
    assert L.dtype == torch.float32 and Bm.dtype == torch.float32 and Bm.dim() == 2 and Bm.stride(1) == 1
    k = L.shape[0]
    assert Bm.shape[1] == k
    M = Bm.shape[0]
    _check(lib().grass_fim_apply(_ptr(L), k, L.stride(0) if k > 1 else 1, _ptr(Bm), M,
                                 Bm.stride(0) if M > 1 else max(k, 1), _stream()), "grass_fim_apply")
    return Bm


def grass_sjlt_table(k: int, s: int, seed: int, kprime: int, device="cuda"):
    """(bucket uint32, sign int8) of length kprime*s, computed by the device hash code."""
    bucket = torch.empty(kprime * s, dtype=torch.int32, device=device)
    sign = torch.empty(kprime * s, dtype=torch.int8, device=device)
    spec = SjltSpec(k, s, seed & 0xFFFFFFFFFFFFFFFF)
    _check(lib().grass_sjlt_table(ctypes.byref(spec), kprime, _ptr(bucket), _ptr(sign), _stream()),
           "grass_sjlt_table")
    return bucket, sign


def grass_validate_mask(idx: torch.Tensor, p: int) -> bool:
    """True if idx (CUDA uint32/int32) is strictly ascending and < p.  Synchronises."""
    _need_cuda(idx)
    code = lib().grass_validate_mask(_ptr(idx), idx.numel(), p, _stream())
    if code == 2:
        return False
    _check(code, "grass_validate_mask")
    return True


def grass_random_mask_host(p: int, kprime: int, seed: int) -> np.ndarray:
    """Random Mask indices (ascending uint32 numpy array), sampled on the host by the library."""
    idx = np.empty(kprime, dtype=np.uint32)
    _check(lib().grass_random_mask_host(p, kprime, seed & 0xFFFFFFFFFFFFFFFF,
                                        idx.ctypes.data_as(ctypes.c_void_p)), "grass_random_mask_host")
    return idx


def mask_to_device(idx: np.ndarray, device="cuda") -> torch.Tensor:
    """uint32 index list -> CUDA tensor holding the same 32-bit patterns."""
    return torch.from_numpy(np.ascontiguousarray(idx, dtype=np.uint32).view(np.int32)).to(device)
