"""Pins for the oracle's indexer score and its prefill/decode drivers.

Each test fixes the result by something other than the oracle's own formula:
a case worked by hand, a special case that collapses to one BLAS matrix
product, closed forms for rank-1 and one-hot inputs, the gate on all-negative
dot products, and invariants that any correct implementation must keep.
Score definition: Sec. 2.1 (multi-head ReLU-gated dot product over preceding
tokens); selection: Sec. 3 "Notation".
"""
import numpy as np
import pytest
import torch

import oracle
from tests.util import bf16_codes_from_f64, codes, f32
from paper_2603_12201_b200 import synth


def _bf(a):
    return bf16_codes_from_f64(a)


def test_hand_worked_case():
    # L = 3 tokens, H = 2 heads, d = 2. All numbers are small integers or halves.
    k = _bf([[1, 0], [0, 1], [1, -1]])
    q = _bf([[[1, 2], [-1, 0]],
             [[2, -1], [0, 3]],
             [[1, 1], [-2, 1]]])
    w = np.array([[0.5, 2.0], [1.0, -1.0], [-0.5, 0.25]], dtype=np.float32)
    # row 0: s=0: h0 1*1+2*0 = 1 -> 0.5*1; h1 -1 -> gated          => 0.5
    # row 1: s=0: h0 2 -> 1*2; h1 0 -> 0                           => 2
    #        s=1: h0 -1 -> gated; h1 3 -> -1*3                     => -3
    # row 2: s=0: h0 1 -> -0.5; h1 -2 -> gated                     => -0.5
    #        s=1: h0 1 -> -0.5; h1 1 -> 0.25                       => -0.25
    #        s=2: h0 0; h1 -3 -> gated                             => 0
    want = np.array([[0.5, -np.inf, -np.inf], [2.0, -3.0, -np.inf], [-0.5, -0.25, 0.0]])
    scores, tk = oracle.indexer_prefill(q, k, w, k_top=2)
    assert np.array_equal(scores, want)
    assert tk.tolist() == [[0, -1], [0, 1], [1, 2]]
    _, tk1 = oracle.indexer_prefill(q, k, w, k_top=1)
    assert tk1.tolist() == [[0], [0], [2]]


def test_nonnegative_inputs_reduce_to_one_matrix_product():
    # With q, k >= 0 every dot product is >= 0, the gate is the identity and
    # I = (sum_h w[t,h] q[t,h,:]) K^T : a single FP64 GEMM.
    L, H, d = 37, 4, 16
    g = torch.Generator().manual_seed(3)
    q = torch.randn(L, H, d, generator=g).abs().to(torch.bfloat16)
    k = torch.randn(L, d, generator=g).abs().to(torch.bfloat16)
    w = torch.randn(L, H, generator=g)
    scores, _ = oracle.indexer_prefill(codes(q), codes(k), f32(w), k_top=4)
    qd, kd, wd = q.to(torch.float64).numpy(), k.to(torch.float64).numpy(), w.to(torch.float64).numpy()
    qbar = (wd[:, :, None] * qd).sum(axis=1)
    want = qbar @ kd.T
    for t in range(L):
        assert np.allclose(scores[t, : t + 1], want[t, : t + 1], rtol=1e-12, atol=1e-12)
        assert np.all(np.isneginf(scores[t, t + 1:]))


def test_rank_one_closed_form():
    # q[t,h,:] = a[t,h] u, k[s,:] = b[s] u  =>  I[t,s] = |u|^2 sum_h w[t,h] max(a[t,h] b[s], 0)
    L, H = 9, 3
    u = np.array([1.0, -2.0, 0.5, 3.0])
    rng = np.random.default_rng(5)
    a = rng.choice([-2.0, -1.0, -0.5, 0.5, 1.0, 2.0], size=(L, H))
    b = rng.choice([-4.0, -1.0, 0.25, 1.0, 2.0], size=L)
    w = rng.standard_normal((L, H)).astype(np.float32)
    q = _bf(a[:, :, None] * u)
    k = _bf(b[:, None] * u)
    scores, _ = oracle.indexer_prefill(q, k, w, k_top=2)
    uu = float(u @ u)
    for t in range(L):
        for s in range(t + 1):
            want = uu * sum(float(w[t, h]) * max(a[t, h] * b[s], 0.0) for h in range(H))
            assert scores[t, s] == pytest.approx(want, rel=1e-13, abs=1e-13)


def test_one_hot_inputs_pick_single_weights():
    # q[t,h,:] = e_{i(t,h)}, k[s,:] = e_{j(s)}  =>  I[t,s] = sum of w[t,h] over heads with i(t,h) == j(s)
    L, H, d = 12, 4, 5
    rng = np.random.default_rng(11)
    i_th = rng.integers(0, d, size=(L, H))
    j_s = rng.integers(0, d, size=L)
    q = np.zeros((L, H, d))
    k = np.zeros((L, d))
    for t in range(L):
        k[t, j_s[t]] = 1.0
        for h in range(H):
            q[t, h, i_th[t, h]] = 1.0
    w = rng.standard_normal((L, H)).astype(np.float32)
    scores, _ = oracle.indexer_prefill(_bf(q), _bf(k), w, k_top=3)
    for t in range(L):
        for s in range(t + 1):
            want = sum(float(w[t, h]) for h in range(H) if i_th[t, h] == j_s[s])
            assert scores[t, s] == pytest.approx(want, abs=1e-15)


def test_gate_zeroes_all_negative_products_and_ties_go_to_lowest_index():
    L, H, d, k_top = 20, 2, 8, 6
    g = torch.Generator().manual_seed(1)
    q = torch.randn(L, H, d, generator=g).abs().to(torch.bfloat16)
    k = (-torch.randn(L, d, generator=g).abs()).to(torch.bfloat16)
    w = torch.randn(L, H, generator=g)
    scores, tk = oracle.indexer_prefill(codes(q), codes(k), f32(w), k_top=k_top)
    for t in range(L):
        assert np.all(scores[t, : t + 1] == 0.0)
        kk = min(k_top, t + 1)
        assert tk[t, :kk].tolist() == list(range(kk))
        assert np.all(tk[t, kk:] == -1)


def test_duplicate_keys_tie_break():
    # keys 2 and 5 are identical and carry the largest score; with k = 1 only the lower index fits
    L, H, d = 8, 2, 4
    q = np.ones((L, H, d))
    k = np.zeros((L, d))
    k[:, 0] = [0.5, 0.25, 4.0, 1.0, 2.0, 4.0, 3.0, 0.125]
    w = np.ones((L, H), dtype=np.float32)
    _, tk = oracle.indexer_prefill(_bf(q), _bf(k), w, k_top=1)
    assert tk[:, 0].tolist() == [0, 0, 2, 2, 2, 2, 2, 2]
    _, tk2 = oracle.indexer_prefill(_bf(q), _bf(k), w, k_top=2)
    assert tk2[7].tolist() == [2, 5] and tk2[4].tolist() == [2, 4]


def _small_case(seed=0, L=48, H=4, d=16, fp8=False):
    return synth.prefill_inputs(L, H, d, seed=seed, fp8=fp8)


@pytest.mark.parametrize("fp8", [False, True])
def test_invariants_causality_short_rows_scaling_head_permutation(fp8):
    inp = _small_case(fp8=fp8)
    dt = oracle.FP8_E4M3 if fp8 else oracle.BF16
    L, H, _ = inp.q.shape
    k_top = 8
    qs, ks = f32(inp.q_scale), f32(inp.k_scale)
    scores, tk = oracle.indexer_prefill(codes(inp.q), codes(inp.k), f32(inp.w), k_top, dt, qs, ks)
    for t in range(L):
        sel = tk[t][tk[t] >= 0]
        assert np.all(sel <= t) and np.all(np.diff(sel) > 0)          # causal, ascending, unique
        assert len(sel) == min(k_top, t + 1)
        if t + 1 <= k_top:
            assert sel.tolist() == list(range(t + 1))                 # short rows take everything
    # positive scaling of w leaves every index set unchanged
    _, tk_s = oracle.indexer_prefill(codes(inp.q), codes(inp.k), f32(inp.w) * 4.0, k_top, dt, qs, ks)
    assert np.array_equal(tk, tk_s)
    # permuting heads together with w leaves scores unchanged up to summation order
    perm = [2, 0, 3, 1]
    sc_p, _ = oracle.indexer_prefill(codes(inp.q)[:, perm], codes(inp.k), f32(inp.w)[:, perm], k_top, dt, qs, ks)
    fin = np.isfinite(scores)
    assert np.allclose(scores[fin], sc_p[fin], rtol=1e-12, atol=1e-12)


def test_fp8_scales_multiply_decoded_codes():
    # non-negative special case again, now through codes * per-token scale
    L, H, d = 21, 2, 8
    g = torch.Generator().manual_seed(9)
    q8, qs = synth.quantize_e4m3(torch.randn(L, H, d, generator=g).abs())
    k8, ks = synth.quantize_e4m3(torch.randn(L, d, generator=g).abs())
    w = torch.randn(L, H, generator=g)
    scores, _ = oracle.indexer_prefill(codes(q8), codes(k8), f32(w), 4, oracle.FP8_E4M3, f32(qs), f32(ks))
    qd = q8.to(torch.float64).numpy() * qs.to(torch.float64).numpy()[:, None, None]
    kd = k8.to(torch.float64).numpy() * ks.to(torch.float64).numpy()[:, None]
    want = (w.to(torch.float64).numpy()[:, :, None] * qd).sum(axis=1) @ kd.T
    for t in range(L):
        assert np.allclose(scores[t, : t + 1], want[t, : t + 1], rtol=1e-12, atol=1e-14)


def test_row_subset_and_chunked_equal_full():
    inp = _small_case(seed=2, L=40)
    q, k, w = codes(inp.q), codes(inp.k), f32(inp.w)
    sc, tk = oracle.indexer_prefill(q, k, w, 5)
    rows = [0, 7, 39, 13]
    sc_r, tk_r = oracle.indexer_prefill(q, k, w, 5, rows=rows)
    assert np.array_equal(sc_r, sc[rows]) and np.array_equal(tk_r, tk[rows])
    # a query chunk [16, 32) against the whole K gives the same rows
    sc_c, tk_c = oracle.indexer_prefill(q[16:32], k, w[16:32], 5, q_begin=16)
    assert np.array_equal(sc_c, sc[16:32]) and np.array_equal(tk_c, tk[16:32])


def test_decode_equals_prefill_row_and_permuted_keys_permute_indices():
    inp = _small_case(seed=4, L=33)
    q, k, w = codes(inp.q), codes(inp.k), f32(inp.w)
    sc, tk = oracle.indexer_prefill(q, k, w, 6)
    # decode for sequences that are prefixes of the same cache: lens = t+1, query = q[t]
    ts = [0, 5, 32]
    offs = np.zeros(len(ts), dtype=np.int64)
    lens = np.array([t + 1 for t in ts], dtype=np.int32)
    sc_d, tk_d = oracle.indexer_decode(q[ts], k, w[ts], offs, lens, 6)
    for j, t in enumerate(ts):
        assert np.array_equal(sc_d[j, : t + 1], sc[t, : t + 1])
        assert np.array_equal(tk_d[j], tk[t])
    # a second cache holding the keys in reversed order selects the mirrored positions
    n = 33
    k2 = np.concatenate([k, k[::-1]], axis=0)
    sc2, tk2 = oracle.indexer_decode(q[[32, 32]], k2, w[[32, 32]], np.array([0, n]), np.array([n, n], dtype=np.int32), 6)
    assert np.array_equal(sc2[1], sc2[0][::-1])
    a = set(tk2[0].tolist())
    b = set((n - 1 - tk2[1]).tolist())
    assert a == b                                   # no exact ties in random data
