"""ctypes loader for the CPU oracle (``grass_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by the tests, by the smoke check and by the
benchmark's CPU-baseline / reference legs.  The CUDA package never imports it
and it never imports the CUDA package.

Arrays are numpy.  bf16 data is passed as ``uint16`` bit patterns together with
``dtype="bf16"``; fp32 data as ``float32`` with ``dtype="f32"``.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "grass_oracle.c")
_SO = os.path.join(_HERE, "libgrass_oracle.so")

F32, BF16 = 0, 1
_DT = {"f32": F32, "bf16": BF16}


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2 -fopenmp) next to its source."""
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < os.path.getmtime(_SRC):
        tmp = _SO + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _SO)
    return _SO


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u64, u32, i64, i32, vp = (ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int64,
                                  ctypes.c_int32, ctypes.c_void_p)
        L.oracle_mix64.restype = u64
        L.oracle_mix64.argtypes = [u64]
        L.oracle_sjlt_hash.restype = u64
        L.oracle_sjlt_hash.argtypes = [u64, u32, u64, u32]
        L.oracle_sjlt_table.restype = None
        L.oracle_sjlt_table.argtypes = [u32, u32, u64, i64, vp, vp]
        L.oracle_random_mask.restype = ctypes.c_int
        L.oracle_random_mask.argtypes = [i64, i64, u64, vp]
        L.oracle_grass.restype = ctypes.c_int
        L.oracle_grass.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, i64, u32, u32, u64, vp, vp]
        L.oracle_factgrass.restype = ctypes.c_int
        L.oracle_factgrass.argtypes = [vp, vp, ctypes.c_int, i32, i32, i32, i32, vp, i32, vp, i32,
                                       u32, u32, u64, vp, vp]
        L.oracle_factgrass_varlen.restype = ctypes.c_int
        L.oracle_factgrass_varlen.argtypes = [vp, vp, ctypes.c_int, i32, i32, i32, vp, i32, vp, i32, u32, u32, u64,
                                              vp, vp, vp, vp]
        L.oracle_score.restype = ctypes.c_int
        L.oracle_score.argtypes = [vp, i64, i64, vp, i64, i64, i64, vp, vp]
        L.oracle_mask.restype = ctypes.c_int
        L.oracle_mask.argtypes = [vp, ctypes.c_int, i64, i64, i64, vp, i64, vp]
        L.oracle_factmask.restype = ctypes.c_int
        L.oracle_factmask.argtypes = [vp, vp, ctypes.c_int, i32, i32, i32, i32, vp, i32, vp, i32, vp, vp]
        L.oracle_fim.restype = ctypes.c_int
        L.oracle_fim.argtypes = [vp, i64, i64, i64, vp, vp]
        L.oracle_fim_solve.restype = ctypes.c_int
        L.oracle_fim_solve.argtypes = [vp, i64, ctypes.c_double, vp, i64, vp]
        L.oracle_num_threads.restype = ctypes.c_int
        L.oracle_set_num_threads.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _check_data(x: np.ndarray, dtype: str) -> None:
    want = np.float32 if dtype == "f32" else np.uint16
    if x.dtype != want or not x.flags.c_contiguous:
        raise ValueError(f"expected C-contiguous {want} array for dtype {dtype}, got {x.dtype}")


def mix64(x: int) -> int:
    return int(lib().oracle_mix64(x & 0xFFFFFFFFFFFFFFFF))


def sjlt_hash(seed: int, s: int, j: int, r: int) -> int:
    return int(lib().oracle_sjlt_hash(seed & 0xFFFFFFFFFFFFFFFF, s, j, r))


def sjlt_table(k: int, s: int, seed: int, kprime: int):
    """(bucket uint32[kprime*s], sign int8[kprime*s]) of the SJLT matrix: input
    position j, draw r -> row bucket[j*s+r] with entry sign[j*s+r]/sqrt(s)."""
    bucket = np.empty(kprime * s, dtype=np.uint32)
    sign = np.empty(kprime * s, dtype=np.int8)
    lib().oracle_sjlt_table(k, s, seed & 0xFFFFFFFFFFFFFFFF, kprime, _ptr(bucket), _ptr(sign))
    return bucket, sign


def random_mask(p: int, kprime: int, seed: int) -> np.ndarray:
    idx = np.empty(kprime, dtype=np.uint32)
    rc = lib().oracle_random_mask(p, kprime, seed & 0xFFFFFFFFFFFFFFFF, _ptr(idx))
    if rc:
        raise ValueError(f"oracle_random_mask failed ({rc})")
    return idx


def grass(g: np.ndarray, idx, k: int, s: int, seed: int, dtype: str = "f32", p=None,
          want_absum: bool = True):
    """GraSS on n dense rows.  g: (n, ld).  Returns (out float64 (n,k), absum or None)."""
    _check_data(g, dtype)
    n, ld = g.shape
    p = ld if p is None else p
    if idx is not None:
        idx = np.ascontiguousarray(idx, dtype=np.uint32)
        kprime = idx.size
    else:
        kprime = p
    out = np.empty((n, k), dtype=np.float64)
    ab = np.empty((n, k), dtype=np.float64) if want_absum else None
    rc = lib().oracle_grass(_ptr(g), _DT[dtype], n, p, ld, _ptr(idx), kprime, k, s,
                            seed & 0xFFFFFFFFFFFFFFFF, _ptr(out), _ptr(ab))
    if rc:
        raise ValueError(f"oracle_grass failed ({rc})")
    return out, ab


def factgrass(A: np.ndarray, G: np.ndarray, mask_in, mask_out, k: int, s: int, seed: int,
              dtype: str = "bf16", want_absum: bool = True):
    """FactGraSS on one linear layer.  A: (B,T,d_in), G: (B,T,d_out)."""
    _check_data(A, dtype)
    _check_data(G, dtype)
    B, T, d_in = A.shape
    B2, T2, d_out = G.shape
    assert (B, T) == (B2, T2)
    mask_in = np.ascontiguousarray(mask_in, dtype=np.uint32)
    mask_out = np.ascontiguousarray(mask_out, dtype=np.uint32)
    out = np.empty((B, k), dtype=np.float64)
    ab = np.empty((B, k), dtype=np.float64) if want_absum else None
    rc = lib().oracle_factgrass(_ptr(A), _ptr(G), _DT[dtype], B, T, d_in, d_out, _ptr(mask_in),
                                mask_in.size, _ptr(mask_out), mask_out.size, k, s,
                                seed & 0xFFFFFFFFFFFFFFFF, _ptr(out), _ptr(ab))
    if rc:
        raise ValueError(f"oracle_factgrass failed ({rc})")
    return out, ab


def factgrass_varlen(A: np.ndarray, G: np.ndarray, mask_in, mask_out, k: int, s: int, seed: int,
                     tok_begin, tok_count, dtype: str = "bf16", want_absum: bool = True):
    """FactGraSS with per-sample sequence lengths.  A: (rows, d_in), G: (rows, d_out); sample b
    owns rows tok_begin[b] .. tok_begin[b] + tok_count[b] - 1."""
    _check_data(A, dtype)
    _check_data(G, dtype)
    assert A.ndim == 2 and G.ndim == 2 and A.shape[0] == G.shape[0]
    tok_begin = np.ascontiguousarray(tok_begin, dtype=np.int64)
    tok_count = np.ascontiguousarray(tok_count, dtype=np.int32)
    B = tok_begin.size
    assert tok_count.size == B
    if B:
        assert tok_begin.min() >= 0 and tok_count.min() >= 0 and int((tok_begin + tok_count).max()) <= A.shape[0]
    mask_in = np.ascontiguousarray(mask_in, dtype=np.uint32)
    mask_out = np.ascontiguousarray(mask_out, dtype=np.uint32)
    out = np.empty((B, k), dtype=np.float64)
    ab = np.empty((B, k), dtype=np.float64) if want_absum else None
    rc = lib().oracle_factgrass_varlen(_ptr(A), _ptr(G), _DT[dtype], B, A.shape[1], G.shape[1], _ptr(mask_in),
                                       mask_in.size, _ptr(mask_out), mask_out.size, k, s,
                                       seed & 0xFFFFFFFFFFFFFFFF, _ptr(tok_begin), _ptr(tok_count), _ptr(out),
                                       _ptr(ab))
    if rc:
        raise ValueError(f"oracle_factgrass_varlen failed ({rc})")
    return out, ab


def score(train: np.ndarray, test: np.ndarray, want_absum: bool = True):
    """scores[i, m] = <train[i], test[m]> in float64."""
    _check_data(train, "f32")
    _check_data(test, "f32")
    N, D = train.shape
    M, D2 = test.shape
    assert D == D2
    sc = np.empty((N, M), dtype=np.float64)
    ab = np.empty((N, M), dtype=np.float64) if want_absum else None
    rc = lib().oracle_score(_ptr(train), N, D, _ptr(test), M, D, D, _ptr(sc), _ptr(ab))
    if rc:
        raise ValueError(f"oracle_score failed ({rc})")
    return sc, ab


def mask(g: np.ndarray, idx, dtype: str = "f32", p=None) -> np.ndarray:
    """Stand-alone Mask: out[i, j] = g[i, idx[j]] (float64)."""
    _check_data(g, dtype)
    n, ld = g.shape
    p = ld if p is None else p
    idx = np.ascontiguousarray(idx, dtype=np.uint32)
    out = np.empty((n, idx.size), dtype=np.float64)
    rc = lib().oracle_mask(_ptr(g), _DT[dtype], n, p, ld, _ptr(idx), idx.size, _ptr(out))
    if rc:
        raise ValueError(f"oracle_mask failed ({rc})")
    return out


def factmask(A: np.ndarray, G: np.ndarray, mask_in, mask_out, dtype: str = "bf16", want_absum: bool = True):
    """Factorised Mask for one linear layer: the k'_in x k'_out block, flattened input-major."""
    _check_data(A, dtype)
    _check_data(G, dtype)
    B, T, d_in = A.shape
    d_out = G.shape[2]
    assert G.shape[:2] == (B, T)
    mask_in = np.ascontiguousarray(mask_in, dtype=np.uint32)
    mask_out = np.ascontiguousarray(mask_out, dtype=np.uint32)
    kp = mask_in.size * mask_out.size
    out = np.empty((B, kp), dtype=np.float64)
    ab = np.empty((B, kp), dtype=np.float64) if want_absum else None
    rc = lib().oracle_factmask(_ptr(A), _ptr(G), _DT[dtype], B, T, d_in, d_out, _ptr(mask_in), mask_in.size,
                               _ptr(mask_out), mask_out.size, _ptr(out), _ptr(ab))
    if rc:
        raise ValueError(f"oracle_factmask failed ({rc})")
    return out, ab


def fim(X: np.ndarray, want_absum: bool = True):
    """Projected Fisher information matrix F = X^T X / n of n compressed gradients (rows of X, float32)."""
    _check_data(X, "f32")
    n, k = X.shape
    F = np.empty((k, k), dtype=np.float64)
    ab = np.empty((k, k), dtype=np.float64) if want_absum else None
    rc = lib().oracle_fim(_ptr(X), n, k, k, _ptr(F), _ptr(ab))
    if rc:
        raise ValueError(f"oracle_fim failed ({rc})")
    return F, ab


def fim_solve(F: np.ndarray, lam: float, Bm: np.ndarray) -> np.ndarray:
    """Rows x_m = (F + lam I)^-1 b_m for the rows b_m of Bm (float64)."""
    F = np.ascontiguousarray(F, dtype=np.float64)
    Bm = np.ascontiguousarray(Bm, dtype=np.float64)
    k = F.shape[0]
    assert F.shape == (k, k) and Bm.shape[1] == k
    X = np.empty_like(Bm)
    rc = lib().oracle_fim_solve(_ptr(F), k, float(lam), _ptr(Bm), Bm.shape[0], _ptr(X))
    if rc == 2:
        raise np.linalg.LinAlgError("F + lambda I is not positive definite")
    if rc:
        raise ValueError(f"oracle_fim_solve failed ({rc})")
    return X


def num_threads() -> int:
    return int(lib().oracle_num_threads())


def set_num_threads(n: int) -> None:
    lib().oracle_set_num_threads(int(n))
