"""Host-side logic that needs no GPU: the tolerance rule itself and the staged / in-place plan of the host-buffer calls."""
import numpy as np
import pytest
import torch

from parity import C_FLOOR, assert_accurate, check_close


def test_tolerance_rule_floor_and_relative_term():
    ref = np.array([100.0, 1e-3, 0.0, -50.0])
    absum = np.array([100.0, 400.0, 0.0, 50.0])
    chain, eps = 4096, 2.0 ** -24
    floor = C_FLOOR * np.sqrt(chain) * eps * absum
    ok = ref + np.array([0.9e-4 * 100.0, 0.9 * floor[1], 0.0, -0.9e-4 * 50.0])
    check_close(ok, ref, absum, 1e-4, chain, eps)
    for j, bump in ((0, 1.2e-4 * 100.0), (1, 1.2 * floor[1]), (3, 1.2e-4 * 50.0)):
        bad = ok.copy()
        bad[j] = ref[j] + bump
        with pytest.raises(AssertionError):
            check_close(bad, ref, absum, 1e-4, chain, eps)
    # the floor is the square-root one: the old worst-case floor (chain * eps * absum) would have let this pass
    bad = ok.copy()
    bad[1] = ref[1] + 0.5 * chain * eps * absum[1]
    with pytest.raises(AssertionError):
        check_close(bad, ref, absum, 1e-4, chain, eps)
    # empty bins must be exactly zero; non-finite references must stay non-finite
    with pytest.raises(AssertionError):
        check_close(ref + np.array([0, 0, 1e-30, 0]), ref, absum, 1e-4, chain, eps)
    with pytest.raises(AssertionError):
        check_close(np.array([1.0]), np.array([np.nan]), np.array([1.0]), 1e-4, 8)
    check_close(np.array([np.nan]), np.array([np.nan]), np.array([1.0]), 1e-4, 8)


def test_assert_accurate_is_relative_to_the_largest_reference():
    ref = np.array([1000.0, 1.0])
    assert_accurate(ref + np.array([0.0, 0.01]), ref, 2e-5)          # 1e-5 of the largest reference
    with pytest.raises(AssertionError):
        assert_accurate(ref + np.array([0.0, 0.03]), ref, 2e-5)


def test_touched_fraction_and_host_plan():
    from paper_2505_18976_b200 import host_api
    # bf16 rows of 4,096 elements = 128 pieces of 32 elements: 64 indices in 64 different pieces touch half the row
    idx = np.arange(64, dtype=np.uint32) * 64
    assert host_api.touched_fraction(idx, 4096, 2) == pytest.approx(0.5)
    assert host_api.touched_fraction(np.arange(4096, dtype=np.uint32), 4096, 2) == 1.0
    # unpinned tensors are never read in place: every tensor is copied, the bytes moved are all bytes
    A = torch.zeros((2, 8, 4096), dtype=torch.bfloat16)
    G = torch.zeros((2, 8, 1024), dtype=torch.bfloat16)
    layer = dict(A=A, G=G, mask_in=idx, mask_out=np.arange(64, dtype=np.uint32), k=16, s=1, seed=0, out_offset=0)
    plan, moved = host_api.factgrass_host_plan([[layer]])
    assert plan == [(False, False)]
    assert moved == A.numel() * 2 + G.numel() * 2
    assert not host_api.factgrass_in_place([[layer]])
