"""Pins for the oracle's Top-k (Sec. 3 "Notation": T_t = Top-k(I_t)), with the
readings: ties to the lowest index, ascending output, -1 padding."""
import numpy as np
import pytest

import oracle


def test_closed_forms_window_and_sink():
    n, k = 50, 7
    inc = np.arange(n, dtype=np.float64) * 0.5 - 3.0
    assert oracle.topk(inc, k).tolist() == list(range(n - k, n))        # increasing scores: the last k
    assert oracle.topk(-inc, k).tolist() == list(range(k))              # decreasing scores: the first k
    assert oracle.topk(np.zeros(n), k).tolist() == list(range(k))       # all equal: the lowest indices


def test_short_rows_are_padded():
    assert oracle.topk(np.array([3.0, 1.0, 2.0]), 5).tolist() == [0, 1, 2, -1, -1]
    assert oracle.topk(np.array([], dtype=np.float64), 3).tolist() == [-1, -1, -1]


def test_against_stable_library_sort():
    rng = np.random.default_rng(0)
    for n, k in [(1, 1), (17, 4), (300, 64), (2000, 256), (2049, 2048)]:
        s = np.round(rng.standard_normal(n) * 4) / 4                    # many exact ties
        kk = min(n, k)
        want = np.sort(np.argsort(-s, kind="stable")[:kk])              # stable: equal scores keep index order
        got = oracle.topk(s, k)
        assert np.array_equal(got[:kk], want) and np.all(got[kk:] == -1)


def test_brute_force_repeated_argmax():
    rng = np.random.default_rng(1)
    for _ in range(50):
        n = int(rng.integers(1, 12))
        k = int(rng.integers(1, 6))
        s = rng.integers(-2, 3, size=n).astype(np.float64)
        left = list(range(n))
        picked = []
        for _ in range(min(k, n)):
            best = left[0]
            for i in left:                                              # first maximum = lowest index on ties
                if s[i] > s[best]:
                    best = i
            picked.append(best)
            left.remove(best)
        got = oracle.topk(s, k)
        assert got[: len(picked)].tolist() == sorted(picked)


def test_negative_zero_equals_positive_zero():
    s = np.array([-0.0, 0.0, -1.0, 0.0])
    assert oracle.topk(s, 2).tolist() == [0, 1]


def test_bad_arguments():
    with pytest.raises(ValueError):
        oracle.topk(np.zeros(3), 0)
