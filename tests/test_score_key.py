"""The tree-build kernel compares fp64 path scores as 64-bit integers through
key = bits ^ ((bits >> 63) & 0x7FFF...F) after storing zero as +0.  This pins, in numpy, what its source
claims: the map keeps order and equality of finite doubles, is its own inverse, and `key - 1` is never
a wrap-around for a finite double (so "at least" can be tested as "above key - 1")."""
import numpy as np

MASK = np.int64(0x7FFFFFFFFFFFFFFF)


def score_key(s: np.ndarray) -> np.ndarray:
    bits = (s + 0.0).view(np.int64)
    return bits ^ ((bits >> np.int64(63)) & MASK)


def key_score(k: np.ndarray) -> np.ndarray:
    return (k ^ ((k >> np.int64(63)) & MASK)).view(np.float64)


def test_order_equality_inverse():
    rng = np.random.default_rng(11)
    s = np.concatenate([
        -np.abs(rng.standard_normal(20000)) * 50.0,          # log-probability sums
        -np.exp(rng.uniform(-700, 5, 20000)),                  # tiny to large magnitudes, denormals included
        np.array([0.0, -0.0, -5e-324, -1e-310, -1.7e308, 1.0, 5e-324, 1.7e308]),
        np.nextafter(-3.25, [-np.inf, np.inf]), np.array([-3.25, -3.25]),
    ])
    k = score_key(s)
    order_f = np.argsort(s, kind="stable")
    assert np.all(np.diff(k[order_f]) >= 0)                    # same order
    i, j = rng.integers(0, len(s), 200000), rng.integers(0, len(s), 200000)
    assert np.array_equal(s[i] < s[j], k[i] < k[j])
    assert np.array_equal(s[i] == s[j], k[i] == k[j])           # -0.0 == +0.0 included
    back = key_score(k)
    assert np.array_equal(back, s + 0.0) and not np.any(np.signbit(back[s == 0.0]))
    assert np.all(k > np.iinfo(np.int64).min + 1)              # key - 1 stays in range
