"""Tolerance rule shared by the parity tests (not a test module).

A compressed output is a signed sum.  With ref_j the oracle's float64 value and
absum_j the same sum over absolute values, the GPU value passes if

    |gpu_j - ref_j| <= max(tol * |ref_j|, C * sqrt(chain) * eps * absum_j),   C = 2

tol   = 1e-4 for fp32 inputs, 2e-2 for bf16 inputs (max relative error per output);
chain = number of fp32 additions that can feed one output (longest accumulation
        chain), eps = 2^-24 for IEEE fp32 adds, 2^-23 where the sum runs inside
        tensor-core accumulators (they truncate).

The second term is the floor below which a relative error is not defined because the
output cancelled.  Every addition of the chain rounds by at most eps times a partial
sum, and no partial sum exceeds absum; `chain` such errors of independent sign add up
like a random walk, sqrt(chain) * eps * absum, and C = 2 leaves two standard
deviations of that crude over-estimate (the partial sums of a cancelling sum are far
below absum).  The worst-case bound, chain * eps * absum, is sqrt(chain) / 2 times
wider: at chain = 4,096 it would let an error of 1 % of a typical score pass.  A
dropped term, a wrong sign or a wrong bucket errs by about absum / load, and a
dropped partial product of a split fp32 operand by 2^-16 absum / sqrt(chain): the
first is caught by this rule at any size, the second by `assert_accurate` below.
Outputs whose absum is zero (empty bins) must be exactly 0.0f.
"""
import numpy as np

C_FLOOR = 2.0


def check_close(gpu, ref, absum, tol, chain, eps=2.0 ** -24, what=""):
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    absum = np.asarray(absum, dtype=np.float64)
    assert gpu.shape == ref.shape == absum.shape, (gpu.shape, ref.shape, absum.shape)
    finite = np.isfinite(ref)
    bound = np.maximum(tol * np.abs(ref), C_FLOOR * np.sqrt(chain) * eps * absum)
    err = np.abs(gpu - ref)
    bad = finite & ~(err <= bound)
    if bad.any():
        i = np.argmax(np.where(bad, err / np.maximum(bound, 1e-300), 0))
        raise AssertionError(f"{what}: {bad.sum()} of {bad.size} outputs out of tolerance; worst at flat {i}: "
                             f"gpu={gpu.flat[i]!r} ref={ref.flat[i]!r} absum={absum.flat[i]!r} bound={bound.flat[i]!r}")
    empty = finite & (absum == 0)
    assert np.all(gpu[empty] == 0.0), f"{what}: empty bins must be exactly zero"
    # non-finite reference values (NaN/Inf inputs) must stay non-finite
    assert np.all(~np.isfinite(gpu[~finite])), f"{what}: NaN/Inf did not propagate"
    well = finite & (np.abs(ref) >= 2.0 ** -10 * absum) & (absum > 0)
    rel = float((err[well] / np.abs(ref[well])).max()) if well.any() else 0.0
    return rel


def assert_accurate(gpu, ref, limit, what=""):
    """Largest error over the largest reference magnitude: the accuracy of the arithmetic itself, free of
    cancellation.  Returns the figure."""
    gpu = np.asarray(gpu, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    fig = float(np.abs(gpu - ref).max() / np.abs(ref).max())
    assert fig <= limit, f"{what}: max|err| / max|ref| = {fig:.3e} exceeds {limit:.1e}"
    return fig


def max_bin_load(bucket, k):
    return int(np.bincount(np.asarray(bucket, dtype=np.int64), minlength=k).max())
