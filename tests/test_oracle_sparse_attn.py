"""Pins for the sparse-attention oracle (Sec. 2.1: attention over the selected subset only; Fig. 2 SparseAttn)."""
import math

import numpy as np
import pytest
import torch

from oracle import sparse_attn
from tests.util import bf16_codes_from_f64, codes


def _rand_bf16(rng, shape, sigma=1.0):
    t = torch.as_tensor(rng.standard_normal(shape) * sigma).to(torch.bfloat16)
    return codes(t), t.to(torch.float64).numpy()


def test_hand_case():
    # one head, d_qk = 2, d_v = 1; two selected rows with scores 0 and ln 3 -> p = (1/4, 3/4)
    ln3 = 1.09375                       # exactly representable in bf16; p = 1/(1+e^ln3), e^ln3/(1+e^ln3)
    q = bf16_codes_from_f64(np.array([[[0.0, 1.0]]]))
    kv = bf16_codes_from_f64(np.array([[2.0, 0.0], [7.0, 5.0], [-4.0, ln3]]))   # row 1 is not selected
    topk = np.array([[0, 2, -1, -1]], dtype=np.int32)
    out, lse = sparse_attn.sparse_attention(q, kv, topk, d_v=1, scale=1.0)
    e = math.exp(ln3)
    assert out[0, 0, 0] == pytest.approx((2.0 - 4.0 * e) / (1.0 + e), rel=1e-14)
    assert lse[0, 0] == pytest.approx(math.log(1.0 + e), rel=1e-14)


def test_full_selection_is_dense_causal_attention():
    # T_t = {0..t}: the definition reduces to textbook causal attention, computed here by the library routine
    rng = np.random.default_rng(5)
    L, H, d_qk, d_v = 24, 3, 16, 8
    qb, q = _rand_bf16(rng, (L, H, d_qk))
    kb, kv = _rand_bf16(rng, (L, d_qk))
    topk = np.full((L, L), -1, dtype=np.int32)
    for t in range(L):
        topk[t, : t + 1] = np.arange(t + 1)
    scale = 0.37
    out, _ = sparse_attn.sparse_attention(qb, kb, topk, d_v, scale)
    qt = torch.as_tensor(q).permute(1, 0, 2)[None]                       # [1, H, L, d]
    kt = torch.as_tensor(kv)[None, None].expand(1, H, L, d_qk)
    vt = torch.as_tensor(kv[:, :d_v])[None, None].expand(1, H, L, d_v)
    ref = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True, scale=scale)
    np.testing.assert_allclose(out, ref[0].permute(1, 0, 2).numpy(), rtol=1e-10, atol=1e-12)


def test_brute_force_loops():
    rng = np.random.default_rng(11)
    n_q, H, d_qk, d_v, n_kv, k = 3, 2, 4, 3, 9, 5
    qb, q = _rand_bf16(rng, (n_q, H, d_qk))
    kb, kv = _rand_bf16(rng, (n_kv, d_qk))
    topk = np.array([[1, 4, 8, -1, -1], [0, 2, 3, 5, 7], [6, -1, -1, -1, -1]], dtype=np.int32)
    scale = 0.5
    out, lse = sparse_attn.sparse_attention(qb, kb, topk, d_v, scale)
    for t in range(n_q):
        sel = [int(j) for j in topk[t] if j >= 0]
        for h in range(H):
            s = [scale * sum(q[t, h, i] * kv[j, i] for i in range(d_qk)) for j in sel]
            z = sum(math.exp(x) for x in s)
            for c in range(d_v):
                want = sum(math.exp(x) / z * kv[j, c] for x, j in zip(s, sel))
                assert out[t, h, c] == pytest.approx(want, rel=1e-12, abs=1e-14)
            assert lse[t, h] == pytest.approx(math.log(z), rel=1e-12)


def test_closed_forms():
    rng = np.random.default_rng(2)
    H, d_qk, d_v, n_kv = 4, 8, 4, 12
    kb, kv = _rand_bf16(rng, (n_kv, d_qk))
    sel = np.array([[1, 3, 4, 9, 11, -1]], dtype=np.int32)
    valid = sel[0][sel[0] >= 0]
    # q = 0: uniform weights -> plain mean of the selected value rows; lse = log(#selected)
    q0 = np.zeros((1, H, d_qk), dtype=np.uint16)
    out, lse = sparse_attn.sparse_attention(q0, kb, sel, d_v, 1.0)
    np.testing.assert_allclose(out[0], np.broadcast_to(kv[valid, :d_v].mean(axis=0), (H, d_v)), rtol=1e-14)
    np.testing.assert_allclose(lse[0], math.log(len(valid)), rtol=1e-14)
    # identical selected rows: the output is that row's value whatever the query
    same = np.repeat(kb[2:3], n_kv, axis=0)
    qb, _ = _rand_bf16(rng, (1, H, d_qk))
    out, _ = sparse_attn.sparse_attention(qb, same, sel, d_v, 0.9)
    np.testing.assert_allclose(out[0], np.broadcast_to(kv[2, :d_v], (H, d_v)), rtol=1e-13)
    # a very large scale picks the value row of the best-scoring selected key
    qb, q = _rand_bf16(rng, (1, H, d_qk))
    out, _ = sparse_attn.sparse_attention(qb, kb, sel, d_v, 4096.0)
    best = valid[np.argmax(q[0] @ kv[valid].T, axis=1)]
    np.testing.assert_allclose(out[0], kv[best, :d_v], rtol=1e-9, atol=1e-12)


def test_invariances():
    rng = np.random.default_rng(3)
    n_q, H, d_qk, d_v, n_kv, k = 4, 3, 8, 4, 40, 10
    qb, q = _rand_bf16(rng, (n_q, H, d_qk))
    kb, kv = _rand_bf16(rng, (n_kv, d_qk))
    topk = np.stack([np.sort(rng.choice(n_kv, k, replace=False)) for _ in range(n_q)]).astype(np.int32)
    topk[1, 6:] = -1
    out, lse = sparse_attn.sparse_attention(qb, kb, topk, d_v, 0.3)
    # the order of the selected set does not matter, nor where the unused slots sit
    perm = np.stack([rng.permutation(row) for row in topk])
    out_p, lse_p = sparse_attn.sparse_attention(qb, kb, perm, d_v, 0.3)
    np.testing.assert_allclose(out_p, out, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse_p, lse, rtol=1e-12)
    # rows outside the selection do not matter
    kb2 = kb.copy()
    unused = np.setdiff1d(np.arange(n_kv), topk[0][topk[0] >= 0])
    kb2[unused] = 0x7FC0        # NaN
    out2, _ = sparse_attn.sparse_attention(qb, kb2, topk, d_v, 0.3, rows=[0])
    np.testing.assert_allclose(out2[0], out[0], rtol=0, atol=0)
    # base offsets: indices relative to a sequence's first cache row
    base = np.array([0, 3, 0, 5], dtype=np.int64)
    absolute = np.where(topk >= base[:, None], topk, -1).astype(np.int32)       # drop entries before the base row
    rel = np.where(absolute >= 0, absolute - base[:, None], -1).astype(np.int32)
    out_r, _ = sparse_attn.sparse_attention(qb, kb, rel, d_v, 0.3, kv_base=base)
    out_a, _ = sparse_attn.sparse_attention(qb, kb, absolute, d_v, 0.3)
    np.testing.assert_allclose(out_r, out_a, rtol=0, atol=0)


def test_shift_of_the_score_only_columns_leaves_the_output_unchanged():
    # adding one vector c to every key in the columns beyond d_v adds scale * <q_h, c> to all scores of head h:
    # the softmax, hence the output, must not move and lse moves by exactly that amount. All values are
    # multiples of 1/8 small enough to stay exact in bf16.
    rng = np.random.default_rng(9)
    H, d_qk, d_v, n_kv = 3, 8, 4, 20
    q = rng.integers(-16, 17, (1, H, d_qk)) / 8.0
    kv = rng.integers(-40, 41, (n_kv, d_qk)) / 8.0
    c = np.zeros(d_qk)
    c[d_v:] = np.array([4, -8, 16, 2]) / 8.0
    topk = np.array([[0, 3, 5, 6, 11, 17, 19, -1]], dtype=np.int32)
    qb = bf16_codes_from_f64(q)
    out, lse = sparse_attn.sparse_attention(qb, bf16_codes_from_f64(kv), topk, d_v, 0.25)
    out_s, lse_s = sparse_attn.sparse_attention(qb, bf16_codes_from_f64(kv + c), topk, d_v, 0.25)
    np.testing.assert_allclose(out_s, out, rtol=1e-12, atol=1e-14)
    np.testing.assert_allclose(lse_s - lse, 0.25 * (q[0] @ c)[None, :], rtol=1e-12, atol=1e-13)


def test_empty_selection():
    qb = np.zeros((2, 2, 4), dtype=np.uint16)
    kb = np.zeros((3, 4), dtype=np.uint16)
    topk = np.array([[-1, -1], [0, -1]], dtype=np.int32)
    out, lse = sparse_attn.sparse_attention(qb, kb, topk, 2, 1.0)
    assert np.all(out[0] == 0) and np.all(np.isneginf(lse[0]))
    assert np.all(lse[1] == 0.0)


def test_entries_that_name_no_cache_row_select_nothing():
    # an entry past the end of the cache (or, with a sequence base, before its start) is padding: the result equals the
    # one with those entries removed, and a query whose entries all fall outside gets out = 0, lse = -inf
    rng = np.random.default_rng(17)
    n_kv, H, d_qk, d_v = 12, 2, 8, 4
    qb, _ = _rand_bf16(rng, (3, H, d_qk))
    kb, _ = _rand_bf16(rng, (n_kv, d_qk))
    dirty = np.array([[3, 12, 7, 500, -1, 0], [12, 13, 99, -1, -1, -1], [11, 2 ** 30, 5, -1, 12, 1]], dtype=np.int32)
    clean = np.array([[3, 7, 0, -1, -1, -1], [-1, -1, -1, -1, -1, -1], [11, 5, 1, -1, -1, -1]], dtype=np.int32)
    out_d, lse_d = sparse_attn.sparse_attention(qb, kb, dirty, d_v, 0.3)
    out_c, lse_c = sparse_attn.sparse_attention(qb, kb, clean, d_v, 0.3)
    assert np.array_equal(out_d, out_c) and np.array_equal(lse_d, lse_c)
    assert np.all(out_d[1] == 0) and np.all(np.isneginf(lse_d[1]))
    # with a base offset the test is on the row actually named: base + entry
    base = np.array([4, 10, 0], dtype=np.int64)
    rel = np.array([[0, 7, 8, -1, -1, -1], [1, 2, 5, -1, -1, -1], [0, 11, 12, -1, -1, -1]], dtype=np.int32)
    rel_clean = np.array([[0, 7, -1, -1, -1, -1], [1, -1, -1, -1, -1, -1], [0, 11, -1, -1, -1, -1]], dtype=np.int32)
    a = sparse_attn.sparse_attention(qb, kb, rel, d_v, 0.3, kv_base=base)
    b = sparse_attn.sparse_attention(qb, kb, rel_clean, d_v, 0.3, kv_base=base)
    assert np.array_equal(a[0], b[0]) and np.array_equal(a[1], b[1])
