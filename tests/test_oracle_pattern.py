"""Pins for the pattern-tooling oracle (Appendix A overlap, Appendix C similarity DP, Algorithm 1)."""
import numpy as np
import pytest

from oracle import pattern, schedule


def test_overlap_closed_forms():
    k = 8
    a = np.array([[0, 1, 2, 3, 4, 5, 6, 7], [0, 2, 4, 6, 8, 10, 12, 14], [0, 1, 2, -1, -1, -1, -1, -1]], dtype=np.int32)
    b = np.array([[0, 1, 2, 3, 4, 5, 6, 7], [1, 3, 5, 7, 9, 11, 13, 15], [1, 2, 3, -1, -1, -1, -1, -1]], dtype=np.int32)
    r = pattern.overlap_rows(a, b)
    assert r.tolist() == [1.0, 0.0, 2.0 / 3.0]                  # identical, disjoint, 2 of 3 valid entries
    assert pattern.overlap(a, a) == 1.0
    assert pattern.overlap(a, b) == pytest.approx((1.0 + 0.0 + 2.0 / 3.0) / 3)
    # sliding windows shifted by s share k - s positions
    w0 = np.arange(100, 100 + k, dtype=np.int32)[None]
    for s in range(k + 1):
        assert pattern.overlap(w0, w0 + s) == pytest.approx((k - s) / k)


def test_dp_objective_on_hand_cases():
    # 4 layers, M = 2: patterns FFSS, FSFS, FSSF
    S = np.zeros((4, 4))
    S[1, 0], S[2, 0], S[3, 0] = 0.9, 0.5, 0.1
    S[2, 1], S[3, 1] = 0.8, 0.7
    S[3, 2] = 0.95
    assert pattern.pattern_value("FFSS", S) == pytest.approx(0.8 + 0.7)
    assert pattern.pattern_value("FSFS", S) == pytest.approx(0.9 + 0.95)
    assert pattern.pattern_value("FSSF", S) == pytest.approx(0.9 + 0.5)
    v, p = pattern.best_pattern_bruteforce(S, 2)
    assert p == "FSFS" and v == pytest.approx(1.85)
    # M = N: nothing is shared; M = 1: everything shares layer 0
    assert pattern.best_pattern_bruteforce(S, 4) == (0.0, "FFFF")
    v1, p1 = pattern.best_pattern_bruteforce(S, 1)
    assert p1 == "FSSS" and v1 == pytest.approx(1.5)


def test_greedy_with_additive_loss_picks_the_cheapest_layers():
    # if the loss is a sum of per-layer costs of the Shared layers, Algorithm 1 flips layers in order of cost
    N, K = 9, 5
    cost = np.array([0.0, 0.7, 0.1, 0.9, 0.3, 0.2, 0.8, 0.05, 0.6])

    def loss(p):
        return float(sum(cost[l] for l, ch in enumerate(p) if ch == "S"))

    pat, order, evals = pattern.greedy_select(N, K, loss)
    assert order == [7, 2, 5, 4, 8]
    assert pat == "FFSFSSFSS" and pat[0] == "F"
    assert evals == sum(N - 1 - s for s in range(K))
    # a full search from all-F to all-S (K = N - 1) performs N(N-1)/2 evaluations, as Sec. 3.1.2 states
    _, _, full = pattern.greedy_select(N, N - 1, loss)
    assert full == N * (N - 1) // 2
    schedule.validate(pat)


def test_greedy_depends_on_the_current_pattern():
    # a loss that penalises runs of Shared layers: the greedy choice changes with what was flipped before
    def loss(p):
        runs = [len(r) for r in p.split("F") if r]
        return float(sum(r * r for r in runs))

    pat, order, _ = pattern.greedy_select(7, 3, loss)
    assert max(len(r) for r in pat.split("F")) == 1           # three isolated Shared layers
    assert order[0] == 1                                       # ties go to the lowest layer
