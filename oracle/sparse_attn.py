"""Oracle for the sparse core attention that consumes the indexer's selection -- TEST INFRASTRUCTURE ONLY.

Sec. 2.1 ("DeepSeek Sparse Attention"): after the lightning indexer has picked the top-k positions T_t, "the
main attention is computed only over this sparse subset", O(L k) instead of O(L^2); Fig. 2 calls the step
SparseAttn_l(X, T^(l)). The paper instantiates it under Multi-head Latent Attention and gives no shapes, so the
reading taken here is the textbook definition restricted to the selected set, in the multi-query form MLA
serves in: every head h of query t attends the same latent rows,

    s[t,h,j] = scale * < q[t,h,:], kv[base_t + T_t[j], 0:d_qk] >            for the usable entries of T_t
    p[t,h,:] = Softmax_j(s[t,h,:])
    out[t,h,:] = sum_j p[t,h,j] * kv[base_t + T_t[j], 0:d_v]                 (values = leading d_v columns of the row)
    lse[t,h]   = log sum_j exp(s[t,h,j])

computed in float64 from the bf16 bit patterns. An entry is usable when T_t[j] >= 0 and the cache row it names,
base_t + T_t[j], exists (lies in [0, n_kv)); the other entries are padding and take no part (reading taken: the paper
only ever forms T_t from cached positions, so an entry that names no row selects nothing). A query without any usable
entry gets out = 0, lse = -inf.
Nothing here is blocked, fused or reordered: gather, one matrix product, a softmax, one matrix product.
"""
from __future__ import annotations

import numpy as np


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> float64: a bf16 is the upper half of a binary32."""
    b = np.ascontiguousarray(bits, dtype=np.uint16)
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def sparse_attention(q_bits, kv_bits, topk, d_v: int, scale: float, kv_base=None, rows=None):
    """q_bits [n_q, H, d_qk] uint16, kv_bits [n_kv, d_qk] uint16, topk [n_q, k] int32 (-1 = unused slot, any order),
    kv_base [n_q] int64 or None (first cache row of the query's sequence). ``rows``: evaluate only these queries.
    Returns (out [n, H, d_v] float64, lse [n, H] float64)."""
    q_bits = np.asarray(q_bits)
    kv = bf16_bits_to_f64(kv_bits)
    n_q, H, d_qk = q_bits.shape
    assert kv.shape[1] == d_qk and 0 < d_v <= d_qk
    rows = np.arange(n_q) if rows is None else np.asarray(rows, dtype=np.int64)
    out = np.zeros((len(rows), H, d_v), dtype=np.float64)
    lse = np.full((len(rows), H), -np.inf, dtype=np.float64)
    for i, t in enumerate(rows):
        sel = np.asarray(topk[t], dtype=np.int64)
        sel = sel[sel >= 0]
        if kv_base is not None:
            sel = sel + int(kv_base[t])
        sel = sel[(sel >= 0) & (sel < kv.shape[0])]           # entries that name no cache row select nothing
        if sel.size == 0:
            continue
        rows_kv = kv[sel]                                   # [n_sel, d_qk]
        s = scale * (bf16_bits_to_f64(q_bits[t]) @ rows_kv.T)   # [H, n_sel]
        m = s.max(axis=1, keepdims=True)
        e = np.exp(s - m)
        z = e.sum(axis=1, keepdims=True)
        out[i] = (e / z) @ rows_kv[:, :d_v]
        lse[i] = (m + np.log(z))[:, 0]
    return out, lse
