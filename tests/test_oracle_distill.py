"""Pins for the distillation-loss oracle (Eq. 1, Eq. 2, Proposition 1)."""
import numpy as np
import pytest

from oracle import distill


def _rand_dist(rng, rows, ld):
    p = rng.random((rows, ld))
    for r in range(rows):
        p[r, r + 1:] = 0.0
        p[r] /= p[r].sum()
    return p


def test_hand_case_and_zero_divergence():
    # two positions, scores (0, ln 3) -> q = (1/4, 3/4); p = (1/2, 1/2): KL = 1/2 ln(2) + 1/2 ln(2/3)
    sc = np.array([[0.0, 0.0], [0.0, np.log(3.0)]])
    p = np.array([[1.0, 0.0], [0.5, 0.5]])
    total, rows = distill.multi_layer_loss(sc, [p])
    assert rows[0] == pytest.approx(0.0, abs=1e-15)            # one causal position: both distributions are (1)
    assert rows[1] == pytest.approx(0.5 * np.log(2.0) + 0.5 * np.log(2.0 / 3.0))
    # KL(q || q) = 0
    q = np.array([[1.0, 0.0], [0.25, 0.75]])
    assert distill.multi_layer_loss(sc, [q])[0] == pytest.approx(0.0, abs=1e-15)
    # scores shifted by a constant give the same distribution
    assert distill.multi_layer_loss(sc + 7.5, [p])[0] == pytest.approx(total)


def test_uniform_closed_form():
    # p uniform on n positions, scores constant -> q uniform -> 0; p one-hot at j -> KL = log n
    n = 9
    sc = np.zeros((n, n))
    p_uni = np.zeros((n, n))
    p_hot = np.zeros((n, n))
    for r in range(n):
        p_uni[r, : r + 1] = 1.0 / (r + 1)
        p_hot[r, r // 2] = 1.0
    assert distill.multi_layer_loss(sc, [p_uni])[0] == pytest.approx(0.0, abs=1e-13)
    _, rows = distill.multi_layer_loss(sc, [p_hot])
    assert np.allclose(rows, np.log(np.arange(1, n + 1)))


def test_proposition_1_difference_does_not_depend_on_the_indexer():
    # L_multi - L_avg = (mean entropy terms of the targets) is the same for any scores: equal gradients (Prop. 1)
    rng = np.random.default_rng(0)
    rows = ld = 12
    targets = [_rand_dist(rng, rows, ld) for _ in range(3)]
    diffs = []
    for seed in range(3):
        sc = np.random.default_rng(10 + seed).standard_normal((rows, ld)) * 3
        diffs.append(distill.multi_layer_loss(sc, targets)[0] - distill.avg_target_loss(sc, targets))
    assert diffs[0] == pytest.approx(diffs[1], abs=1e-10) and diffs[1] == pytest.approx(diffs[2], abs=1e-10)
    assert diffs[0] >= -1e-12                                   # Jensen: the mean of KLs is at least the KL of the mean
    # a single target: the two losses coincide
    sc = rng.standard_normal((rows, ld))
    assert distill.multi_layer_loss(sc, targets[:1])[0] == pytest.approx(distill.avg_target_loss(sc, targets[:1]))


def test_topk_restricted_form():
    rng = np.random.default_rng(2)
    rows = ld = 10
    p = _rand_dist(rng, rows, ld)
    sc = rng.standard_normal((rows, ld))
    k = 4
    topk = np.full((rows, k), -1, dtype=np.int32)
    for r in range(rows):
        sel = np.sort(rng.choice(r + 1, size=min(k, r + 1), replace=False))
        topk[r, : len(sel)] = sel
    total, per_row = distill.multi_layer_loss(sc, [p], topk=topk)
    # by hand for one row: restrict, renormalise, KL
    r = 7
    idx = topk[r][topk[r] >= 0]
    pr = p[r, idx] / p[r, idx].sum()
    q = np.exp(sc[r, idx]) / np.exp(sc[r, idx]).sum()
    assert per_row[r] == pytest.approx(float((pr * np.log(pr / q)).sum()))
    # rows whose set is the whole causal prefix equal the unrestricted loss
    full = np.full((rows, rows), -1, dtype=np.int32)
    for r in range(rows):
        full[r, : r + 1] = np.arange(r + 1)
    assert distill.multi_layer_loss(sc, [p], topk=full)[0] == pytest.approx(distill.multi_layer_loss(sc, [p])[0])
