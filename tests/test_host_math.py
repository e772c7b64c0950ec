"""Arithmetic facts the CUDA path relies on, checked on the CPU with numpy (IEEE double and float).

The placement kernel and the optimal-assignment kernel replace the float32 division `tot / n` (n a small
integer) by the double product `tot * (1/n)` rounded to float32; the results must be identical to the
division the oracle performs, bit for bit."""
import numpy as np


def _check(x, n):
    ref = x / np.float32(n)
    got = (x.astype(np.float64) * np.float64(1.0 / n)).astype(np.float32)
    assert np.array_equal(ref.view(np.uint32), got.view(np.uint32)), n


def test_double_product_with_reciprocal_rounds_like_float_division():
    rng = np.random.default_rng(7)
    bits = rng.integers(0, 0x7F7FFFFF, size=400_000, dtype=np.uint32)          # every finite non-negative float
    everywhere = bits.view(np.float32)
    typical = (rng.random(400_000) * 16).astype(np.float32)                     # sums of slowdowns
    # quotients that end just below, at and just above the midpoint of two floats
    m = rng.integers(1 << 23, 1 << 24, size=100_000, dtype=np.int64)
    for n in range(1, 17):
        _check(everywhere, n)
        _check(typical, n)
        for delta in (-1, 0, 1):
            near = ((2 * m + 1) * n // 2 + delta).astype(np.float64)            # about (m + 1/2) * n
            _check(near.astype(np.float32) * np.float32(2.0 ** -20), n)
        small = (rng.integers(1, 1 << 20, size=100_000).astype(np.float32)) * np.float32(2.0 ** -149)   # subnormals
        _check(small, n)
