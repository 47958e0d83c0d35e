"""Host-side pattern tooling of the library (Appendix C similarity DP, Algorithm 1 greedy search) against
the oracle: the DP against enumeration of every pattern, the greedy driver against the oracle's loop."""
import numpy as np
import pytest

from oracle import pattern as opat
from oracle import schedule as osched


@pytest.fixture(scope="module")
def idxc():
    from paper_2603_12201_b200 import build
    build.build()
    from paper_2603_12201_b200 import binding
    return binding


def test_dp_matches_enumeration(idxc):
    rng = np.random.default_rng(0)
    for N in (1, 2, 3, 5, 8, 11):
        S = np.tril(rng.random((N, N)), k=-1)
        for M in range(1, N + 1):
            pat, val = idxc.pattern_search_dp(S, M)
            osched.validate(pat)
            assert pat.count("F") == M
            want_v, _ = opat.best_pattern_bruteforce(S, M)
            assert val == pytest.approx(want_v, abs=1e-12)
            assert opat.pattern_value(pat, S) == pytest.approx(want_v, abs=1e-12)   # the pattern achieves the optimum


def test_dp_hand_case_and_bad_arguments(idxc):
    S = np.zeros((4, 4))
    S[1, 0], S[2, 0], S[3, 0], S[2, 1], S[3, 1], S[3, 2] = 0.9, 0.5, 0.1, 0.8, 0.7, 0.95
    assert idxc.pattern_search_dp(S, 2) == ("FSFS", pytest.approx(1.85))
    with pytest.raises(idxc.IdxcError):
        idxc.pattern_search_dp(S, 0)
    with pytest.raises(idxc.IdxcError):
        idxc.pattern_search_dp(S, 5)


def test_dp_at_the_size_of_the_papers_models(idxc):
    # 47 layers, keep 12 (the 1/4 setting): too many patterns to enumerate; check validity and local optimality
    rng = np.random.default_rng(1)
    N, M = 47, 12
    S = np.tril(rng.random((N, N)), k=-1)
    pat, val = idxc.pattern_search_dp(S, M)
    osched.validate(pat)
    assert pat.count("F") == M and val == pytest.approx(opat.pattern_value(pat, S))
    # moving any single Full layer (not the first) to a neighbouring Shared slot cannot improve the value
    for l in range(1, N):
        for l2 in (l - 1, l + 1):
            if pat[l] == "F" and 1 <= l2 < N and pat[l2] == "S":
                alt = list(pat)
                alt[l], alt[l2] = "S", "F"
                assert opat.pattern_value("".join(alt), S) <= val + 1e-12


def test_greedy_matches_oracle_loop(idxc):
    cost = np.array([0.0, 0.7, 0.1, 0.9, 0.3, 0.2, 0.8, 0.05, 0.6])

    def additive(p):
        return float(sum(cost[l] for l, ch in enumerate(p) if ch == "S"))

    def runs(p):
        return float(sum(len(r) ** 2 for r in p.split("F") if r)) + 0.01 * additive(p)

    for loss in (additive, runs):
        for K in (0, 1, 5, 8):
            got = idxc.pattern_search_greedy(9, K, loss)
            want = opat.greedy_select(9, K, loss)
            assert got == want
    assert idxc.pattern_search_greedy(9, 8, additive)[2] == 9 * 8 // 2       # N(N-1)/2 evaluations for a full search
    # the loss after each step is the loss of the pattern with exactly the layers flipped so far
    pat, order, _, losses = idxc.pattern_search_greedy(9, 5, runs, want_losses=True)
    for step in range(5):
        p = "".join("S" if l in order[: step + 1] else "F" for l in range(9))
        assert losses[step] == pytest.approx(runs(p), rel=1e-15)
    assert pat == "".join("S" if l in order else "F" for l in range(9))
    with pytest.raises(idxc.IdxcError):
        idxc.pattern_search_greedy(9, 9, additive)                            # layer 0 can never be Shared
