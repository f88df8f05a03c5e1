"""Pins for the oracle's priority transform p = (|delta| + eps)^alpha."""
import numpy as np


def _ulp_diff(a, b):
    ia = np.float32(a).view(np.int32).astype(np.int64)
    ib = np.float32(b).view(np.int32).astype(np.int64)
    return abs(int(ia) - int(ib))


def test_matches_libm_pow_within_one_ulp(oracle_mod):
    rng = np.random.default_rng(11)
    n = 60_000
    delta = np.concatenate([rng.normal(size=n // 3), np.exp(2.0 * rng.normal(size=n // 3)),
                            rng.uniform(-1e-4, 1e-4, size=n // 3)]).astype(np.float32)
    alpha = rng.uniform(0.05, 2.0, size=n).astype(np.float32)
    alpha[: n // 2] = np.float32(0.6)
    eps = np.float32(1e-6)
    worst = 0
    for d, a in zip(delta, alpha):
        got = oracle_mod.priority_pow(d, eps, a)
        y = np.float32(np.abs(d) + eps)
        want = np.float32(np.power(np.float64(y), np.float64(a)))
        assert got is not None
        worst = max(worst, _ulp_diff(got, want))
        assert abs(float(got) - float(want)) <= 1e-6 * float(want)
    assert worst <= 1     # binary64 evaluation rounded once: at most a double-rounding ulp


def test_exact_cases(oracle_mod):
    for y in [1.0, 0.75, 3.0, 1e-6, 12345.678, 2.0**-100, 2.0**100]:
        assert oracle_mod.priority_pow(y, 0.0, 1.0) == np.float32(y)          # alpha = 1
    for n in range(-30, 31):
        assert oracle_mod.priority_pow(4.0**n, 0.0, 0.5) == np.float32(2.0**n)    # square root of 4^n
        assert oracle_mod.priority_pow(2.0**n, 0.0, 2.0) == np.float32(4.0**n)    # square of 2^n
        assert oracle_mod.priority_pow(-(2.0**n), 0.0, 2.0) == np.float32(4.0**n)  # |delta|
    assert oracle_mod.priority_pow(3.0, 1.0, 0.5) == np.float32(2.0)           # eps is added first
    assert oracle_mod.priority_pow(123.0, 1e-6, 0.0) == np.float32(1.0)        # alpha = 0
    assert oracle_mod.priority_pow(0.0, 0.0, 0.6) == np.float32(0.0)           # y = 0


def test_invalid_entries(oracle_mod):
    assert oracle_mod.priority_pow(float("nan"), 1e-6, 0.6) is None
    assert oracle_mod.priority_pow(float("inf"), 1e-6, 0.6) is None
    assert oracle_mod.priority_pow(-float("inf"), 1e-6, 0.6) is None
    assert oracle_mod.priority_pow(3e38, 3e38, 0.6) is None      # |delta| + eps overflows binary32
    assert oracle_mod.priority_pow(1e30, 0.0, 2.0) is None       # result overflows binary32
    assert oracle_mod.priority_pow(1e-30, 0.0, 2.0) == np.float32(0.0)   # underflows to zero


def test_monotone_in_delta(oracle_mod):
    ys = np.sort(np.abs(np.random.default_rng(3).normal(size=5000)).astype(np.float32))
    ps = np.array([oracle_mod.priority_pow(y, 1e-6, 0.6) for y in ys])
    assert np.all(np.diff(ps) >= 0)
