"""Oracle for the pattern tooling on index tensors -- TEST INFRASTRUCTURE ONLY.

* overlap: the top-k index overlap |T^(i) n T^(j)| / k of Appendix A, per query row and averaged.
  Reading: a row with fewer than k valid entries (short causal rows, -1 padding) is divided by its
  number of valid entries, so that identical rows give 1.
* similarity DP of Appendix C: among the patterns with exactly M Full layers (the first layer Full),
  maximise sum over Shared layers l of S[l, src(l)]. Written here as the definition itself: enumerate
  every pattern (small N only). The recurrence printed in the appendix reuses the letter k and carries a
  stray condition on c_j; the objective above is what it solves.
* greedy layer selection, Algorithm 1: K steps; each step tries every remaining Full layer (never the
  first) as Shared, keeps the one with the lowest loss. Ties go to the lowest layer (the paper is silent).
"""
from __future__ import annotations

import itertools

import numpy as np

from . import schedule


def overlap_rows(Ta: np.ndarray, Tb: np.ndarray) -> np.ndarray:
    """Per-row overlap ratio of two index tensors [rows, k] (ascending, -1 padded)."""
    assert Ta.shape == Tb.shape
    out = np.zeros(Ta.shape[0], dtype=np.float64)
    for r in range(Ta.shape[0]):
        a = Ta[r][Ta[r] >= 0]
        b = Tb[r][Tb[r] >= 0]
        out[r] = len(np.intersect1d(a, b)) / len(a) if len(a) else 0.0
    return out


def overlap(Ta: np.ndarray, Tb: np.ndarray) -> float:
    return float(overlap_rows(Ta, Tb).mean()) if Ta.shape[0] else 0.0


def pattern_value(pattern: str, S: np.ndarray) -> float:
    """Objective of Appendix C: total similarity of the Shared layers to their source layers."""
    src = schedule.source_layers(pattern)
    return float(sum(S[l, src[l]] for l in range(len(pattern)) if pattern[l] == "S"))


def best_pattern_bruteforce(S: np.ndarray, M: int):
    """All patterns with exactly M Full layers and a Full first layer; returns (best value, one best pattern)."""
    N = S.shape[0]
    best_v, best_p = -np.inf, None
    for rest in itertools.combinations(range(1, N), M - 1):
        fl = {0, *rest}
        p = "".join("F" if l in fl else "S" for l in range(N))
        v = pattern_value(p, S)
        if v > best_v:
            best_v, best_p = v, p
    return best_v, best_p


def greedy_select(N: int, K: int, eval_loss):
    """Algorithm 1. eval_loss(pattern) -> float. Returns (pattern, order of flipped layers, evaluations)."""
    c = ["F"] * N
    remaining = list(range(1, N))          # layer 0 (the paper's layer 1) is always Full
    order, evals = [], 0
    for _ in range(K):
        best_l, best_loss = None, None
        for l in remaining:
            trial = c.copy()
            trial[l] = "S"
            loss = eval_loss("".join(trial))
            evals += 1
            if best_loss is None or loss < best_loss:
                best_l, best_loss = l, loss
        c[best_l] = "S"
        remaining.remove(best_l)
        order.append(best_l)
    return "".join(c), order, evals
