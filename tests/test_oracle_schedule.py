"""Pins for the schedule oracle: the pattern strings the paper prints
(Appendix B), the definition f(l) = max{j < l : c_j = F} evaluated with a
library string search, and the properties Sec. 3 "Overview" states."""
import os

import numpy as np
import pytest

from oracle import schedule

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "searched_patterns.txt")


def printed_patterns():
    out = []
    with open(GOLDEN) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            model, frac, n, pat = line.split()
            out.append((model, frac, int(n), pat))
    return out


def test_printed_patterns_are_well_formed():
    pats = printed_patterns()
    assert len(pats) == 5
    for model, frac, n, pat in pats:
        assert len(pat) == n and set(pat) <= {"F", "S"}
        assert pat[0] == "F"                                # "The first layer is always F"
        schedule.validate(pat)
    counts = {(m, f): p.count("F") for m, f, _, p in pats}
    # kept indexers: about N/2, N/4, N/8 of the 47 layers; 40 and 22 of GLM-5's 78
    assert counts[("GLM-4.7-Flash-30B", "1/2")] == 24
    assert counts[("GLM-4.7-Flash-30B", "1/4")] == 12
    assert counts[("GLM-4.7-Flash-30B", "1/8")] == 7
    assert counts[("GLM-5", "1/2")] == 40
    assert counts[("GLM-5", "1/4")] == 22


def test_source_layers_match_library_search_on_printed_patterns():
    for _, _, n, pat in printed_patterns():
        src = schedule.source_layers(pat)
        for l in range(n):
            want = l if pat[l] == "F" else pat.rfind("F", 0, l)
            assert src[l] == want
        # the 1/4 pattern of the 30B model keeps these layers (0-based), read off the printed string
    p14 = [p for m, f, _, p in printed_patterns() if m.startswith("GLM-4.7") and f == "1/4"][0]
    assert [i for i, c in enumerate(p14) if c == "F"] == [0, 2, 4, 9, 13, 16, 17, 20, 23, 28, 32, 37]


def test_run_shares_bit_for_bit_and_counts_calls():
    pat = "FSSFSFSS"
    rng = np.random.default_rng(0)
    fresh = [rng.integers(0, 100, size=(4, 3)).astype(np.int32) for _ in pat]
    called = []

    def indexer(l):
        called.append(l)
        return fresh[l]

    out, calls = schedule.run(pat, indexer)
    assert calls == pat.count("F") and called == [0, 3, 5]          # S layers never run their indexer
    src = schedule.source_layers(pat)
    for l in range(len(pat)):
        assert np.array_equal(out[l], fresh[src[l]])
        assert out[l] is out[src[l]]                                 # reuse, not recomputation


def test_all_full_is_standard_dsa():
    out, calls = schedule.run("FFFF", lambda l: l * 10)
    assert out == [0, 10, 20, 30] and calls == 4


@pytest.mark.parametrize("bad", ["", "SFF", "FXS", "fss"])
def test_invalid_patterns(bad):
    with pytest.raises(ValueError):
        schedule.validate(bad)
