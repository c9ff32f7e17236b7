"""Pins of the oracle's round-to-nearest-even into fp32 / fp16 / bf16 (CPU only).

The sweeps round once per sweep to the storage type.  The rounding is pinned by brute force (search
of the nearest value in the enumerated table of every finite value of the 16-bit format, ties to the
even significand) and by numpy's own correctly rounded float64 -> float16/float32 casts.
"""
import numpy as np
import pytest

import oracle


def _table(dtype):
    bits = np.arange(65536, dtype=np.uint32).astype(np.uint16)
    vals = oracle.decode(bits, dtype)
    keep = np.isfinite(vals)
    bits, vals = bits[keep], vals[keep]
    order = np.argsort(vals, kind="stable")
    return bits[order], vals[order]


def _brute_nearest(x, bits_tab, vals_tab):
    """Nearest table value; on a tie the one whose bit pattern is even."""
    i = np.searchsorted(vals_tab, x)
    i = np.clip(i, 1, len(vals_tab) - 1)
    lo, hi = vals_tab[i - 1], vals_tab[i]
    dlo, dhi = x - lo, hi - x
    pick_hi = (dhi < dlo) | ((dhi == dlo) & (bits_tab[i] % 2 == 0))
    return np.where(pick_hi, hi, lo)


@pytest.mark.parametrize("dtype", [oracle.BF16, oracle.F16])
def test_rounding_matches_brute_force_nearest(dtype):
    bits_tab, vals_tab = _table(dtype)
    rng = np.random.default_rng(3)
    top = 60000.0 if dtype == oracle.F16 else 1e30
    x = np.concatenate([
        rng.standard_normal(20000) * 0.02,                   # weight-sized
        rng.standard_normal(20000) * 1e-3,                   # perturbation-sized
        rng.uniform(-1, 1, 20000) * top,
        rng.uniform(-1, 1, 5000) * (6e-8 if dtype == oracle.F16 else 1e-38),   # subnormal range
    ])
    # exact midpoints between neighbours (the ties), away from the zero pair
    mids = 0.5 * (vals_tab[:-1] + vals_tab[1:])
    mids = mids[(vals_tab[:-1] != 0) | (vals_tab[1:] != 0)]
    x = np.concatenate([x, mids[:: 7]])
    got = oracle.round_to(x, dtype)
    exp = _brute_nearest(x, bits_tab, vals_tab)
    np.testing.assert_array_equal(got, exp)


def test_fp16_and_fp32_match_numpy_casts():
    rng = np.random.default_rng(4)
    x = np.concatenate([rng.standard_normal(100000) * 0.02, rng.standard_normal(1000) * 1e-6, [0.0, -0.0, 65504.0, 65519.9, 65520.0, 1e-8]])
    with np.errstate(over="ignore"):
        np.testing.assert_array_equal(oracle.round_to(x, oracle.F16), x.astype(np.float16).astype(np.float64))
    np.testing.assert_array_equal(oracle.round_to(x, oracle.F32), x.astype(np.float32).astype(np.float64))


@pytest.mark.parametrize("dtype", [oracle.BF16, oracle.F16, oracle.F32])
def test_encode_decode_roundtrip(dtype):
    rng = np.random.default_rng(6)
    x = rng.standard_normal(5000) * 0.02
    stored = oracle.encode(x, dtype)
    back = oracle.decode(stored, dtype)
    np.testing.assert_array_equal(back, oracle.round_to(x, dtype))
    np.testing.assert_array_equal(oracle.encode(back, dtype), stored)
    if dtype == oracle.F16:
        np.testing.assert_array_equal(stored.view(np.float16).astype(np.float64), back)
    if dtype == oracle.BF16:
        np.testing.assert_array_equal((stored.astype(np.uint32) << 16).view(np.float32).astype(np.float64), back)
