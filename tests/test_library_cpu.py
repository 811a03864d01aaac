"""CPU-side checks of the CUDA library: it loads without a GPU, exports every symbol the
header declares, rejects bad arguments on the host, and its host-side Random Mask sampler
is bit-exact with the oracle."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def cuda_lib():
    from paper_2505_18976_b200 import build, binding
    build.build()
    return binding


def test_exports_every_declared_symbol(cuda_lib):
    hdr = open(os.path.join(ROOT, "include", "grass.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b((?:fact)?grass_[a-z_]+)\s*\(", hdr))
    assert {"grass_compress", "factgrass_compress", "factgrass_compress_grouped", "grass_score"} <= names
    L = cuda_lib.lib()
    for n in names:
        assert hasattr(L, n), f"{n} declared in grass.h but not exported"
    assert names <= set(cuda_lib.EXPORTS) | names


def test_status_strings(cuda_lib):
    L = cuda_lib.lib()
    assert L.grass_status_string(0) == b"ok"
    assert len({L.grass_status_string(i) for i in range(6)}) == 6


def test_host_side_argument_checks_need_no_gpu(cuda_lib):
    L = cuda_lib.lib()
    spec = cuda_lib.SjltSpec(16, 1, 0)
    bad_k = cuda_lib.SjltSpec(0, 1, 0)
    bad_s = cuda_lib.SjltSpec(16, 0, 0)
    one = ctypes.c_void_p(256)   # never dereferenced: the call must fail before any launch
    INVALID, UNSUPPORTED = 1, 3
    assert L.grass_compress(one, 0, 4, 10, 10, None, 10, None, one, 16, None, None) == INVALID
    assert L.grass_compress(one, 0, 4, 10, 10, None, 10, ctypes.byref(bad_k), one, 16, None, None) == INVALID
    assert L.grass_compress(one, 0, 4, 10, 10, None, 10, ctypes.byref(bad_s), one, 16, None, None) == INVALID
    assert L.grass_compress(one, 0, 4, 10, 9, None, 10, ctypes.byref(spec), one, 16, None, None) == INVALID   # ld < p
    assert L.grass_compress(one, 0, 4, 10, 10, one, 11, ctypes.byref(spec), one, 16, None, None) == INVALID   # k' > p
    assert L.grass_compress(one, 0, 4, 10, 10, None, 5, ctypes.byref(spec), one, 16, None, None) == INVALID   # identity needs k'=p
    assert L.grass_compress(one, 0, 4, 10, 10, None, 10, ctypes.byref(spec), one, 15, None, None) == INVALID  # ld_out < k
    assert L.grass_compress(one, 0, -1, 10, 10, None, 10, ctypes.byref(spec), one, 16, None, None) == INVALID
    assert L.grass_compress(one, 7, 4, 10, 10, None, 10, ctypes.byref(spec), one, 16, None, None) == UNSUPPORTED
    assert L.grass_compress(one, 0, 0, 10, 10, None, 10, ctypes.byref(spec), one, 16, None, None) == 0        # n == 0
    # FactGraSS: an unknown dtype and kin > d_in are invalid
    assert L.factgrass_compress(one, one, 7, 2, 8, 16, 16, one, 4, one, 4, ctypes.byref(spec), one, 16, None, None) == INVALID
    assert L.factgrass_compress(one, one, 1, 2, 8, 16, 16, one, 17, one, 4, ctypes.byref(spec), one, 16, None, None) == INVALID
    assert L.factgrass_compress(one, one, 1, 2, 8, 16, 16, one, 4, one, 4, None, one, 16, None, None) == INVALID
    assert L.factgrass_compress(one, one, 1, 0, 8, 16, 16, one, 4, one, 4, ctypes.byref(spec), one, 16, None, None) == 0
    assert L.factgrass_compress_grouped(None, 1, 1, 2, 8, one, 16, None, 0, None, None) == INVALID
    assert L.grass_score(one, 4, 3, one, 4, 8, 8, one, 4, None) == INVALID      # ld_train < D
    assert L.grass_score(one, 0, 8, one, 4, 8, 8, one, 4, None) == 0
    assert L.grass_random_mask_host(10, 11, 0, None) == INVALID
    assert L.factgrass_grouped_workspace_bytes(224) >= 224 * 64
    assert L.factgrass_grouped_workspace_bytes(224) % 256 == 0


def test_random_mask_host_bit_exact_with_oracle(cuda_lib, oracle_mod):
    for p, kp, seed in ((65536, 8192, 0), (4194304, 65536, 0), (768, 128, 3), (14336, 64, 6), (100, 100, 7),
                        (1000, 1, 8), (50, 0, 1), (12345, 6789, 0xFFFFFFFFFFFFFFFF)):
        a = cuda_lib.grass_random_mask_host(p, kp, seed)
        b = oracle_mod.random_mask(p, kp, seed)
        assert a.dtype == np.uint32 and np.array_equal(a, b), (p, kp, seed)


def test_oracle_and_cuda_path_share_no_code():
    """Neither side imports or includes the other."""
    pkg = os.path.join(ROOT, "paper_2505_18976_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"import\s+oracle|from\s+oracle|grass_oracle|oracle/|oracle\.", src), \
                    f"{f} reaches into the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c", ".h")):
            src = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2505_18976_b200" not in src and "grass.h" not in src and "libgrass_b200" not in src


def test_host_api_chooses_in_place_gather_only_for_sparse_masks():
    """At 64-byte granularity a mask of every 64th fp32 coordinate touches a quarter of the pieces, a mask of every
    4th coordinate touches all of them; unpinned inputs are always staged."""
    import torch
    from paper_2505_18976_b200 import host_api
    assert host_api.touched_fraction(np.arange(0, 4096, 64), 4096, 4) == pytest.approx(0.25)
    assert host_api.touched_fraction(np.arange(0, 4096, 4), 4096, 4) == 1.0
    assert host_api.touched_fraction(np.array([0, 1, 31, 32]), 64, 2) == 1.0
    g = torch.zeros((2, 4096))
    assert not host_api.grass_in_place([g], np.arange(0, 4096, 64))          # not pinned
    assert not host_api.grass_in_place([g], None)
