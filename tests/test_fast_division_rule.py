"""The per-group histogram kernel turns a flat index into (row, offset) with one multiply-high:
n // d == (n * m) >> 32 with m = (2^32 - 1) // d + 1, claimed exact whenever n * d <= 2^32.
Brute force over the divisors and index ranges its units can have."""
import numpy as np


def _quot(n, d):
    if d == 1:
        return n
    m = np.uint64(0xFFFFFFFF // d + 1)
    return (n * m) >> np.uint64(32)


def test_multiply_high_division_is_exact_where_the_kernel_uses_it():
    for d in range(1, 4097):                               # row lengths of the short-row walkers
        top = min((1 << 32) // d, 1 << 18)                 # a unit holds at most 2^17 and a few elements
        n = np.arange(0, top, dtype=np.uint64)
        assert np.array_equal(_quot(n, d), n // np.uint64(d)), d
    rng = np.random.default_rng(7)
    for d in (3, 7, 49, 196, 3136, 12544, 50176, 65535, 65536, 131071):   # long rows, packed runs
        top = (1 << 32) // d
        n = np.unique(np.concatenate([np.arange(max(0, top - 200000), top, dtype=np.uint64),
                                      rng.integers(0, top, 500000, dtype=np.uint64)]))
        assert np.array_equal(_quot(n, d), n // np.uint64(d)), d


def test_multiply_high_division_fails_beyond_its_bound():
    """The bound matters: far past n * d = 2^32 the rule is wrong, so the kernel's range checks are needed."""
    d = 3
    n = np.arange((1 << 32) - 1000, 1 << 32, dtype=np.uint64)
    assert not np.array_equal(_quot(n, d), n // np.uint64(d))
