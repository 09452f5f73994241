"""The tree-build kernel divides indices by the run-time k, k^2 and d through a float reciprocal:
floor((float(e) + 0.5f) * (1.0f / float(d))).  This pins the claim in its source that the result is the
exact integer quotient over the operand range the kernel uses (and well beyond it), with the same
IEEE single-precision operations in numpy."""
import numpy as np


def fast_div(e: np.ndarray, d: int) -> np.ndarray:
    inv = np.float32(1.0) / np.float32(d)
    return np.floor((e.astype(np.float32) + np.float32(0.5)) * inv).astype(np.int64)


def test_exact_over_the_kernels_range():
    # pairs of a level: e < k^3 <= 32768; candidates: e < k + 15 k^2 < 16384; divisors k <= 32, k^2 <= 1024, d <= 16
    e = np.arange(0, 70000, dtype=np.int64)
    for d in range(1, 1025):
        assert np.array_equal(fast_div(e, d), e // d), d


def test_exact_up_to_the_stated_bound():
    rng = np.random.default_rng(7)
    e = np.concatenate([rng.integers(0, 1 << 22, size=200000), np.array([(1 << 22) - 1, (1 << 22) - 1024])])
    for d in list(range(1, 65)) + [100, 127, 128, 255, 256, 511, 512, 1000, 1023, 1024]:
        assert np.array_equal(fast_div(e, d), e // d), d
    # multiples of d and their predecessors are the cases a reciprocal gets wrong first
    for d in (3, 7, 10, 49, 100, 1000, 1023):
        m = np.arange(d, 1 << 22, d, dtype=np.int64)
        assert np.array_equal(fast_div(m, d), m // d), d
        assert np.array_equal(fast_div(m - 1, d), (m - 1) // d), d
