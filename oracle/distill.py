"""Oracle for the multi-layer distillation loss (training-aware IndexCache) -- TEST INFRASTRUCTURE ONLY.

Eq. (1) "multi-layer distillation loss":  L_multi = sum_{j=0..m} 1/(m+1) sum_t KL( p_t^(l+j) || q_t^(l) ),
with q_t = Softmax(I_t) the indexer's output distribution of the Full layer l (Sec. 3 "Notation") and p_t^(l+j)
the aggregated attention distribution of the served layer l+j at position t. Both live on the causal positions
s <= t. Eq. (2): L_avg = sum_t KL( mean_j p_t^(l+j) || q_t ). Sparse-training form (Sec. 3.2 "Training"): the KL
is computed only over the selected top-k tokens; reading taken: p and q are both restricted to T_t and
renormalised over it. 0 * log 0 = 0.
"""
from __future__ import annotations

import numpy as np


def _log_softmax(x: np.ndarray) -> np.ndarray:
    m = x.max()
    return x - (m + np.log(np.exp(x - m).sum()))


def kl_row(p: np.ndarray, scores: np.ndarray) -> float:
    """KL(p || Softmax(scores)) for one row, float64; entries with p == 0 contribute 0."""
    logq = _log_softmax(scores.astype(np.float64))
    p = p.astype(np.float64)
    nz = p > 0
    return float((p[nz] * (np.log(p[nz]) - logq[nz])).sum())


def multi_layer_loss(scores: np.ndarray, targets: list[np.ndarray], first_len: int = 1, len_step: int = 1, topk=None):
    """Returns (L_multi, per-row contribution). scores [rows, ld]; targets: m+1 arrays [rows, ld]; row r uses
    positions [0, first_len + r*len_step). With topk [rows, k] (ascending, -1 padded) the row uses those positions
    only, p renormalised over them."""
    rows = scores.shape[0]
    w = 1.0 / len(targets)
    out = np.zeros(rows, dtype=np.float64)
    for r in range(rows):
        n = first_len + r * len_step
        if topk is None:
            idx = np.arange(n)
        else:
            idx = topk[r][topk[r] >= 0].astype(np.int64)
        s = scores[r, idx]
        for p in targets:
            pr = p[r, idx].astype(np.float64)
            if topk is not None:
                tot = pr.sum()
                pr = pr / tot if tot > 0 else pr
            out[r] += w * kl_row(pr, s)
    return float(out.sum()), out


def avg_target_loss(scores: np.ndarray, targets: list[np.ndarray], first_len: int = 1, len_step: int = 1) -> float:
    """Eq. (2): distillation against the averaged target."""
    pbar = np.mean(np.stack([t.astype(np.float64) for t in targets]), axis=0)
    return multi_layer_loss(scores, [pbar], first_len, len_step)[0]
