"""OS^3 scheduler: the oracle against what the paper and the mathematics fix, then the
library's host functions against the oracle (no GPU involved)."""
import ctypes
import random
from fractions import Fraction

import pytest

from oracle import os3


# ------------------------------------------------------------------ pins of the oracle
@pytest.mark.parametrize("s", [1, 2, 3, 8, 20])
@pytest.mark.parametrize("g", [Fraction(0), Fraction(1, 7), Fraction(3, 5), Fraction(9, 10)])
def test_expected_verified_equals_the_appendix_derivation(s, g):
    """Appendix A.2, first line: 1 + sum_{i=1}^{s-2} i g^i (1-g) + (s-1) g^(s-1), and last line:
    (1 - g^s) / (1 - g), both in exact rational arithmetic (at s = 1 the first line, whose
    trailing term vanishes, is the single verified document)."""
    first = 1 + sum(i * g ** i * (1 - g) for i in range(1, s - 1)) + (s - 1) * g ** (s - 1) if s > 1 else 1
    closed = (1 - g ** s) / (1 - g)
    assert closed == sum(g ** i for i in range(s))
    if s >= 2:
        assert first == closed
    assert abs(os3.expected_verified(float(g), s) - float(closed)) < 1e-12


def test_expected_verified_by_simulation():
    rng = random.Random(5)
    g, s, n = 0.55, 6, 200_000
    total = 0
    for _ in range(n):
        m = 0
        while m < s and rng.random() < g:
            m += 1
        total += min(m + 1, s)           # the corrected document counts as verified
    assert abs(total / n - os3.expected_verified(g, s)) < 0.01


def test_objective_special_cases():
    a, b = 2.0, 7.0
    # gamma = 0: one document per s a + b, so the shortest stride wins
    assert os3.objective(0.0, a, b, 4, False) == pytest.approx(1.0 / (4 * a + b))
    assert os3.best_stride([], [], 0.6, a, b, 16, False) == 1
    # free speculation (a = 0): more speculation never hurts, the largest stride wins
    assert os3.best_stride([3, 3], [3, 3], 0.9, 0.0, b, 12, False) == 12
    # asynchronous verification is never slower, and equal when gamma = 0
    for s in range(1, 9):
        assert os3.latency(0.5, a, b, s, True) <= os3.latency(0.5, a, b, s, False)
        assert os3.latency(0.0, a, b, s, True) == os3.latency(0.0, a, b, s, False)
    # all-match probability 1: latency (s - 1) a + max(a, b)
    assert os3.latency(1.0, a, b, 5, True) == pytest.approx(4 * a + max(a, b))
    # worked value: gamma = 1/2, s = 2, a = 1, b = 2, synchronous: 1.5 documents in 4 time units
    assert os3.objective(0.5, 1.0, 2.0, 2, False) == pytest.approx(0.375)
    # asynchronous, same numbers: latency 1/4 * (1 + 2) + 3/4 * 4 = 3.75
    assert os3.objective(0.5, 1.0, 2.0, 2, True) == pytest.approx(1.5 / 3.75)


def test_gamma_estimate():
    # Appendix A.2: sum M / (sum M + number of steps with a mismatch)
    assert os3.estimate_gamma([3, 1, 0], [3, 3, 2], 1.0) == pytest.approx(4 / (4 + 2))
    assert os3.estimate_gamma([3, 3], [3, 3], 0.6) == 0.6          # all matched: truncated
    assert os3.estimate_gamma([0], [4], 0.6) == 0.0
    assert os3.estimate_gamma([], [], 0.6) == 0.0
    # the estimate is the maximum-likelihood one: it recovers gamma from simulated steps
    rng = random.Random(9)
    g, M, S = 0.4, [], []
    for _ in range(20_000):
        s = rng.randint(1, 8)
        m = 0
        while m < s and rng.random() < g:
            m += 1
        M.append(m)
        S.append(s)
    assert abs(os3.estimate_gamma(M, S, 1.0) - g) < 0.01


def test_best_stride_is_the_exhaustive_argmax():
    # histories whose estimate is exactly 0.2, 0.5 and 0.6: hits / (hits + steps with a mismatch)
    histories = {0.2: ([1, 0, 0, 0], [2, 1, 1, 1]), 0.5: ([1], [2]), 0.6: ([3, 0], [4, 1])}
    for g, (M, S) in histories.items():
        assert os3.estimate_gamma(M, S, 1.0) == pytest.approx(g)
        for a, b in ((1.0, 1.0), (1.0, 10.0), (3.0, 100.0)):
            for async_v in (False, True):
                vals = [os3.objective(g, a, b, s, async_v) for s in range(1, 33)]
                s_best = 1 + max(range(32), key=lambda i: (vals[i], -i))
                assert os3.best_stride(M, S, 1.0, a, b, 32, async_v) == s_best
    # a slower verification step favours a longer stride
    assert os3.best_stride([1], [2], 1.0, 1.0, 50.0, 32, False) > os3.best_stride([1], [2], 1.0, 1.0, 2.0, 32, False)


# ------------------------------------------------------------------ library against the oracle
@pytest.fixture(scope="module")
def lib():
    from paper_2401_14021_b200 import build
    lib = ctypes.CDLL(build.build())
    f64, i32 = ctypes.c_double, ctypes.c_int32
    lib.ralm_os3_expected_verified.restype = f64
    lib.ralm_os3_expected_verified.argtypes = [f64, i32]
    lib.ralm_os3_objective.restype = f64
    lib.ralm_os3_objective.argtypes = [f64, f64, f64, i32, i32]
    lib.ralm_os3_gamma.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(i32), i32, f64, ctypes.POINTER(f64)]
    lib.ralm_os3_stride.argtypes = [ctypes.POINTER(i32), ctypes.POINTER(i32), i32, f64, f64, f64, i32, i32,
                                    ctypes.POINTER(i32)]
    return lib


def test_library_matches_the_oracle(lib):
    rng = random.Random(11)
    for _ in range(300):
        w = rng.randint(0, 5)
        S = [rng.randint(1, 8) for _ in range(w)]
        M = [rng.randint(0, s) for s in S]
        a, b = rng.uniform(0.01, 5.0), rng.uniform(0.01, 50.0)
        async_v = rng.random() < 0.5
        gmax = rng.choice([0.6, 0.9, 1.0])
        arr = (ctypes.c_int32 * max(w, 1))
        m_arr, s_arr = arr(*M) if w else arr(0), arr(*S) if w else arr(1)
        g = ctypes.c_double()
        assert lib.ralm_os3_gamma(m_arr, s_arr, w, gmax, ctypes.byref(g)) == 0
        g_o = os3.estimate_gamma(M, S, gmax)
        assert g.value == pytest.approx(g_o, abs=1e-15)
        for s in (1, 2, 5, 13):
            if g_o < 1.0:
                assert lib.ralm_os3_expected_verified(g_o, s) == pytest.approx(os3.expected_verified(g_o, s), rel=1e-12)
            assert lib.ralm_os3_objective(g_o, a, b, s, int(async_v)) == pytest.approx(
                os3.objective(g_o, a, b, s, async_v), rel=1e-12)
        out = ctypes.c_int32()
        assert lib.ralm_os3_stride(m_arr, s_arr, w, gmax, a, b, 16, int(async_v), ctypes.byref(out)) == 0
        s_o = os3.best_stride(M, S, gmax, a, b, 16, async_v)
        if out.value != s_o:            # only an exact tie of the objective may differ
            assert os3.objective(g_o, a, b, out.value, async_v) == pytest.approx(
                os3.objective(g_o, a, b, s_o, async_v), rel=1e-12)
    assert lib.ralm_os3_expected_verified(1.0, 7) == 7.0


def test_library_argument_errors(lib):
    arr = (ctypes.c_int32 * 2)
    g, out = ctypes.c_double(), ctypes.c_int32()
    assert lib.ralm_os3_gamma(arr(3, 1), arr(2, 2), 2, 0.6, ctypes.byref(g)) == 1      # matched > stride
    assert lib.ralm_os3_gamma(arr(0, 0), arr(0, 2), 2, 0.6, ctypes.byref(g)) == 1      # stride < 1
    assert lib.ralm_os3_gamma(None, None, 2, 0.6, ctypes.byref(g)) == 1
    assert lib.ralm_os3_stride(arr(1, 1), arr(2, 2), 2, 0.6, 1.0, 1.0, 0, 0, ctypes.byref(out)) == 1
    assert lib.ralm_os3_stride(arr(1, 1), arr(2, 2), 2, 0.6, -1.0, 1.0, 8, 0, ctypes.byref(out)) == 1
    assert lib.ralm_os3_stride(None, None, 0, 0.6, 1.0, 1.0, 8, 0, ctypes.byref(out)) == 0 and out.value == 1
