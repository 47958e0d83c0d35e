"""GPU parity: the CUDA path, called through the C-ABI binding, against the FP64 oracle
on the same seeded inputs, element by element. Sizes span several 128-key tiles, several
work items and ragged tails; edge cases cover short rows, chunking, ties and empty input."""
import numpy as np
import pytest
import torch

import oracle
from oracle import schedule as oracle_schedule
from paper_2603_12201_b200 import binding as idxc
from paper_2603_12201_b200 import synth
from tests.util import (RTOL_BF16, RTOL_FP8, assert_scores_close, assert_topk_valid, codes, f32)

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _to_dev(inp):
    for name in ("q", "k", "w", "q_scale", "k_scale", "q_step", "k_cache", "k_offsets", "lens"):
        if hasattr(inp, name) and getattr(inp, name) is not None:
            setattr(inp, name, getattr(inp, name).to(DEV))
    return inp


def _oracle_prefill(inp, k_top, rows=None, q_begin=0, q_slice=None):
    dt = oracle.FP8_E4M3 if inp.fp8 else oracle.BF16
    q, w, qs = inp.q, inp.w, inp.q_scale
    if q_slice is not None:
        q, w = q[q_slice], w[q_slice]
        qs = None if qs is None else qs[q_slice]
    return oracle.indexer_prefill(codes(q), codes(inp.k), f32(w), k_top, dt, f32(qs), f32(inp.k_scale),
                                  q_begin=q_begin, rows=rows)


def _gpu_prefill(inp, k_top, flags=0, with_scores=True, q_begin=0, q_slice=None, workspace=None):
    q, w, qs = inp.q, inp.w, inp.q_scale
    if q_slice is not None:
        q, w = q[q_slice].contiguous(), w[q_slice].contiguous()
        qs = None if qs is None else qs[q_slice].contiguous()
    q_len, L_k = q.shape[0], inp.k.shape[0]
    ld = (L_k + 3) // 4 * 4
    scores = torch.full((q_len, ld), float("nan"), device=DEV) if with_scores else None
    topk = torch.full((q_len, k_top), -7, dtype=torch.int32, device=DEV)
    if workspace is None and not with_scores:
        workspace = idxc.alloc_workspace(idxc.prefill_workspace_bytes(q_len, L_k, q.shape[1], q.shape[2], k_top), DEV)
    idxc.indexer_prefill(q, inp.k, w, k_top, qs, inp.k_scale, q_begin=q_begin, scores_out=scores, topk_out=topk,
                         workspace=workspace, flags=flags)
    idxc.poll_device_status()
    return (None if scores is None else scores.cpu().numpy()), topk.cpu().numpy()


def _check_prefill(inp, k_top, g_scores, g_topk, rtol, rows=None):
    """All rows (or the listed ones) of a full prefill (q_begin = 0) against the oracle.
    Returns the fraction of rows whose index set equals the oracle's exactly."""
    o_scores, _ = _oracle_prefill(inp, k_top, rows=rows)
    row_ids = range(g_topk.shape[0]) if rows is None else rows
    exact = 0
    for j, t in enumerate(row_ids):
        o_row = o_scores[j, : t + 1]
        if g_scores is not None:
            assert_scores_close(g_scores[t, : t + 1], o_row, rtol, what=f"row {t}")
        exact += assert_topk_valid(g_topk[t], o_row, k_top, rtol, what=f"row {t}")
    return exact / max(len(row_ids), 1)


def _own_topk_exact(g_scores, g_topk, k_top, q_begin=0):
    """The selector alone: indices must be the exact top-k (lowest index on ties) of the GPU's own scores."""
    for r in range(g_topk.shape[0]):
        n = q_begin + r + 1
        kk = min(k_top, n)
        order = np.argsort(-g_scores[r, :n].astype(np.float64), kind="stable")
        assert np.array_equal(np.sort(order[:kk]), g_topk[r, :kk]), f"row {r}"
        assert np.all(g_topk[r, kk:] == -1)


# ------------------------------------------------------------------------------ top-k alone
@pytest.mark.parametrize("n,k_top", [(1, 1), (5, 8), (300, 64), (4096, 2048), (4100, 2048), (33000, 2048), (131072, 2048)])
def test_topk_rows_matches_oracle(n, k_top):
    g = torch.Generator().manual_seed(n)
    rows = 6
    ld = (n + 3) // 4 * 4
    s = torch.randn(rows, ld, generator=g)
    s[1] = torch.round(s[1] * 2) / 2                      # many exact ties
    s[2] = 0.0                                            # all equal (threshold bucket overflows)
    s[3] = torch.arange(ld, dtype=torch.float32)          # increasing: sliding window
    s[4] = -torch.arange(ld, dtype=torch.float32)         # decreasing: sink
    s[5, ::3] = -0.0
    lens = torch.tensor([n, n, n, n, n, max(n - 3, 0)], dtype=torch.int32)
    out = torch.full((rows, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.topk_rows(s.to(DEV), k_top, out, lens=lens.to(DEV))
    out = out.cpu().numpy()
    for r in range(rows):
        want = oracle.topk(s[r, : int(lens[r])].to(torch.float64).numpy(), k_top)
        assert np.array_equal(out[r], want), f"row {r}"


def test_topk_rows_many_rows_constant_tied_and_crowded():
    """More than 1024 rows (the many-rows kernel instance) with the rows that defeat the fast path: constant rows,
    heavy ties, and rows whose scores all share their leading key bits, so that the threshold bucket holds the whole
    row and the select has to finish over the row itself. Bit-exact against the oracle, every row."""
    g = torch.Generator().manual_seed(99)
    n_rows, ld, k_top = 1100, 3000, 512
    s = torch.randn(n_rows, ld, generator=g)
    s[::7] = 0.0                                                        # constant rows
    s[1::7] = torch.round(s[1::7] * 2) / 2                              # a handful of distinct values
    s[2::7] = 1.0 + torch.rand(s[2::7].shape, generator=g) * 2.0 ** -6  # one crowded bucket: all in [1, 1.016)
    s[3::7] = -(1.0 + torch.randint(0, 3, s[3::7].shape, generator=g).float() * 2.0 ** -20)   # crowded and tied
    s[4::7, ::2] = -0.0
    s[4::7, 1::2] = 0.0                                                 # -0 == +0
    lens = torch.randint(0, ld + 1, (n_rows,), generator=g, dtype=torch.int32)
    lens[:40] = ld
    out = torch.full((n_rows, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.topk_rows(s.to(DEV), k_top, out, lens=lens.to(DEV))
    out = out.cpu().numpy()
    s64 = s.to(torch.float64).numpy()
    for r in range(n_rows):
        assert np.array_equal(out[r], oracle.topk(s64[r, : int(lens[r])], k_top)), f"row {r}"


def _selected_dominate(scores: torch.Tensor, topk: torch.Tensor, lens: torch.Tensor, k_top: int):
    """Property that holds for any correct selection: per row min(k, len) distinct ascending in-range indices, and no
    unselected score of the row exceeds a selected one (checked on the device over the whole output)."""
    n_rows, ld = scores.shape
    kk = torch.clamp(lens.long(), max=k_top)
    col = torch.arange(k_top, device=scores.device)
    valid = col[None, :] < kk[:, None]
    assert bool(((topk >= 0) == valid).all())
    assert bool((topk[:, 1:] > topk[:, :-1])[valid[:, 1:]].all())
    assert bool((torch.where(valid, topk.long(), torch.zeros_like(topk, dtype=torch.long)) < torch.clamp(lens.long(), min=1)[:, None]).all())
    for r0 in range(0, n_rows, 64):                                     # slabs bound the transient memory
        sl = slice(r0, min(n_rows, r0 + 64))
        sc = scores[sl]
        chosen = torch.zeros_like(sc, dtype=torch.bool)
        idx = torch.where(valid[sl], topk[sl].long(), torch.zeros_like(topk[sl], dtype=torch.long))
        chosen.scatter_(1, idx, valid[sl])
        inside = torch.arange(ld, device=sc.device)[None, :] < lens[sl].long()[:, None]
        lo_sel = torch.where(chosen, sc, torch.full_like(sc, float("inf"))).amin(dim=1)
        hi_rest = torch.where(inside & ~chosen, sc, torch.full_like(sc, float("-inf"))).amax(dim=1)
        assert bool((hi_rest <= lo_sel).all())


@pytest.mark.parametrize("n_rows", [5, 1024])
def test_topk_rows_longer_than_the_selection_map(n_rows):
    """Rows of more than 524288 scores exceed the shared-memory selection map of both one-CTA kernel instances
    (few rows: 1024 threads; 1024 rows and more: 256 threads) and are finished over the row itself."""
    n, k_top = 524288 + 517, 2048
    ld = (n + 3) // 4 * 4
    g = torch.Generator(device=DEV).manual_seed(n_rows)
    s = torch.randn(n_rows, ld, generator=g, device=DEV)
    s[1] = torch.round(s[1] * 4) / 4                                     # ties across the threshold
    s[2] = 0.0
    lens = torch.full((n_rows,), n, dtype=torch.int32, device=DEV)
    lens[3] = n - 5
    out = torch.full((n_rows, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.topk_rows(s, k_top, out, lens=lens)
    _selected_dominate(s, out, lens, k_top)
    for r in sorted({0, 1, 2, 3, n_rows - 1}):
        want = oracle.topk(s[r, : int(lens[r])].to(torch.float64).cpu().numpy(), k_top)
        assert np.array_equal(out[r].cpu().numpy(), want), f"row {r}"


def test_topk_rows_with_masked_entries_read_at_full_length():
    """Rows filled under IDXC_FLAG_FILL_MASKED hold -inf beyond the causal part. Read at full length with fewer than k
    finite scores, the k-th largest is -inf itself: every finite position is selected first, then the lowest masked
    positions; every output slot is written."""
    L, H, d, k_top = 300, 16, 64, 64
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=14))
    ld = 304
    sc = torch.zeros((L, ld), device=DEV)
    idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, scores_out=sc, flags=idxc.FLAG_FILL_MASKED)
    out = torch.full((L, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.topk_rows(sc, k_top, out, first_len=L, len_step=0)
    out = out.cpu().numpy()
    host = sc.cpu().to(torch.float64).numpy()
    for r in range(L):
        assert np.array_equal(out[r], oracle.topk(host[r, :L], k_top)), f"row {r}"
    assert out[10].tolist() == list(range(k_top))                        # 11 finite scores, then masked ones in order


def test_topk_rows_causal_lengths_and_empty():
    g = torch.Generator().manual_seed(5)
    n_rows, ld, k_top = 70, 72, 16
    s = torch.randn(n_rows, ld, generator=g)
    out = torch.full((n_rows, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.topk_rows(s.to(DEV), k_top, out, first_len=1, len_step=1)
    out = out.cpu().numpy()
    for r in range(n_rows):
        assert np.array_equal(out[r], oracle.topk(s[r, : r + 1].to(torch.float64).numpy(), k_top))
    empty = torch.empty((0, 8), device=DEV)
    idxc.topk_rows(empty, 4, torch.empty((0, 4), dtype=torch.int32, device=DEV), first_len=1, len_step=1)


# ------------------------------------------------------------------------------ prefill
@pytest.mark.parametrize("L,H,d,k_top,fp8,flags", [
    (200, 4, 32, 16, False, idxc.FLAG_SIMT_SCORER),
    (200, 4, 32, 16, True, idxc.FLAG_SIMT_SCORER),
    (300, 16, 64, 32, False, 0),
    (517, 32, 64, 64, False, 0),
    (1000, 64, 128, 128, False, 0),
    (700, 32, 128, 64, False, 0),
    (900, 64, 128, 100, True, 0),
    (333, 16, 128, 40, True, 0),
    # the remaining (d_I, H_I, dtype) kernels the library accepts
    (640, 64, 64, 50, False, 0),
    (450, 16, 128, 33, False, 0),
    (520, 32, 128, 77, True, 0),
    # odd sizes around a key tile and a work item
    (1, 64, 128, 4, False, 0),
    (127, 64, 128, 16, False, 0),
    (129, 64, 128, 16, True, 0),
    (2049, 64, 128, 256, False, 0),
])
def test_prefill_matches_oracle(L, H, d, k_top, fp8, flags):
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=10 + L, fp8=fp8))
    g_scores, g_topk = _gpu_prefill(inp, k_top, flags=flags)
    rtol = RTOL_FP8 if fp8 else RTOL_BF16
    _check_prefill(inp, k_top, g_scores, g_topk, rtol)
    _own_topk_exact(g_scores, g_topk, k_top)
    # entries above the diagonal are never written
    iu = np.triu_indices(L, k=1)
    assert np.all(np.isnan(g_scores[:, :L][iu]))


def test_config1_full():
    c = synth.CONFIGS["cfg1"]
    inp = _to_dev(synth.prefill_inputs(c["L"], c["H"], c["d"], seed=c["seed"]))
    g_scores, g_topk = _gpu_prefill(inp, c["k_top"])
    frac = _check_prefill(inp, c["k_top"], g_scores, g_topk, RTOL_BF16)
    _own_topk_exact(g_scores, g_topk, c["k_top"])
    assert frac > 0.98          # near-ties inside the tolerance band are rare


def test_prefill_chunked_workspace_and_scoreless_paths_agree():
    L, H, d, k_top = 1100, 64, 128, 96
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=77))
    s_full, t_full = _gpu_prefill(inp, k_top)
    # no score output: scores go through the workspace; a small workspace forces several chunks
    ld = (L + 31) // 32 * 32
    _, t_ws = _gpu_prefill(inp, k_top, with_scores=False)
    _, t_small = _gpu_prefill(inp, k_top, with_scores=False, workspace=idxc.alloc_workspace(64 * ld * 4, DEV))
    assert np.array_equal(t_ws, t_full) and np.array_equal(t_small, t_full)
    # query chunks against the full K (chunked prefill) give the same rows
    for q0, q1 in [(0, 256), (256, 700), (700, 1100)]:
        s_c, t_c = _gpu_prefill(inp, k_top, q_begin=q0, q_slice=slice(q0, q1))
        assert np.array_equal(t_c, t_full[q0:q1])
        for r in range(q1 - q0):
            assert np.array_equal(s_c[r, : q0 + r + 1], s_full[q0 + r, : q0 + r + 1])
    with pytest.raises(idxc.IdxcError) as e:
        _gpu_prefill(inp, k_top, with_scores=False, workspace=idxc.alloc_workspace(8 * ld * 4, DEV))
    assert e.value.status == idxc.ERR_WORKSPACE


def test_prefill_short_chunk_against_long_context_equals_the_whole_prefill():
    """A few hundred query rows against a long K are cut into runs of key tiles so that every SM gets work; a whole
    prefill of the same length has enough blocks of rows and is not cut. Both must give the same bits."""
    L, H, d, k_top = 20000, 64, 128, 512
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=91))
    s_full, t_full = _gpu_prefill(inp, k_top)
    for q0, q1 in [(19400, 20000), (12345, 12601), (0, 300), (19995, 20000), (7, 8)]:      # (down to a handful of rows)
        s_c, t_c = _gpu_prefill(inp, k_top, q_begin=q0, q_slice=slice(q0, q1))
        assert np.array_equal(t_c, t_full[q0:q1])
        for r in sorted({0, min(1, q1 - q0 - 1), (q1 - q0) // 2, q1 - q0 - 1}):
            assert np.array_equal(s_c[r, : q0 + r + 1], s_full[q0 + r, : q0 + r + 1])
            assert np.all(np.isnan(s_c[r, q0 + r + 1:]))
    # and in e4m3
    inp8 = _to_dev(synth.prefill_inputs(9000, H, d, seed=92, fp8=True))
    s_full, t_full = _gpu_prefill(inp8, k_top)
    s_c, t_c = _gpu_prefill(inp8, k_top, q_begin=8500, q_slice=slice(8500, 9000))
    assert np.array_equal(t_c, t_full[8500:])
    assert np.array_equal(s_c[499, :9000], s_full[8999, :9000])


def test_prefill_duplicate_keys_pick_lowest_index_and_gate():
    L, H, d, k_top = 400, 16, 64, 8
    inp = synth.prefill_inputs(L, H, d, seed=3)
    inp.k[200:] = inp.k[:200]                       # every key appears twice: bit-identical scores
    inp = _to_dev(inp)
    g_scores, g_topk = _gpu_prefill(inp, k_top)
    assert np.array_equal(g_scores[399, 200:400], g_scores[399, :200])
    _own_topk_exact(g_scores, g_topk, k_top)
    _check_prefill(inp, k_top, g_scores, g_topk, RTOL_BF16)
    # all dot products <= 0: every score is exactly zero and the lowest positions win
    inp2 = synth.prefill_inputs(L, H, d, seed=4)
    inp2.q = inp2.q.abs()
    inp2.k = -inp2.k.abs()
    inp2 = _to_dev(inp2)
    s2, t2 = _gpu_prefill(inp2, k_top)
    for t in range(L):
        assert np.all(s2[t, : t + 1] == 0.0)
        kk = min(k_top, t + 1)
        assert t2[t, :kk].tolist() == list(range(kk))


def test_prefill_fill_masked_writes_the_causal_mask():
    # IDXC_FLAG_FILL_MASKED: s > t becomes -inf up to column L_k - 1, the scores s <= t and the columns beyond L_k stay
    # as they are; chunked calls (q_begin > 0) mask relative to the absolute position
    L, H, d, k_top = 333, 16, 64, 16
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=12))
    ld = 352
    plain = torch.full((L, ld), 7.0, device=DEV)
    idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, scores_out=plain)
    filled = torch.full((L, ld), 7.0, device=DEV)
    idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, scores_out=filled, flags=idxc.FLAG_FILL_MASKED)
    t = torch.arange(L, device=DEV)[:, None]
    s_ = torch.arange(ld, device=DEV)[None, :]
    causal, masked, beyond = s_ <= t, (s_ > t) & (s_ < L), s_ >= L
    assert torch.equal(filled[causal.expand(L, ld)], plain[causal.expand(L, ld)])
    assert bool(torch.isneginf(filled[masked.expand(L, ld)]).all())
    assert bool((filled[beyond.expand(L, ld)] == 7.0).all()) and bool((plain[masked.expand(L, ld)] == 7.0).all())
    q0, q1 = 100, 230
    part = torch.full((q1 - q0, ld), 7.0, device=DEV)
    idxc.indexer_prefill(inp.q[q0:q1], inp.k, inp.w[q0:q1], k_top, q_begin=q0, scores_out=part, flags=idxc.FLAG_FILL_MASKED)
    assert torch.equal(part, filled[q0:q1])
    # the masked rows feed a soft-max directly
    assert bool(torch.isfinite(torch.softmax(filled[:, :L], dim=1)).all())


def test_prefill_rejects_bad_arguments():
    inp = _to_dev(synth.prefill_inputs(64, 16, 64, seed=1))
    topk = torch.empty((64, 8), dtype=torch.int32, device=DEV)
    ws = idxc.alloc_workspace(1 << 20, DEV)
    with pytest.raises(idxc.IdxcError) as e:
        idxc.indexer_prefill(inp.q, inp.k, inp.w, 8, q_begin=1, topk_out=topk, workspace=ws)      # L_k < q_begin + q_len
    assert e.value.status == idxc.ERR_INVALID_ARG
    with pytest.raises(idxc.IdxcError) as e:
        idxc.indexer_prefill(inp.q, inp.k, inp.w, 8)                                              # no output at all
    assert e.value.status == idxc.ERR_INVALID_ARG
    with pytest.raises(idxc.IdxcError) as e:
        idxc.indexer_prefill(inp.q, inp.k, inp.w, 8, topk_out=topk)                               # no workspace
    assert e.value.status == idxc.ERR_WORKSPACE
    with pytest.raises(ValueError):
        idxc.indexer_prefill(inp.q.cpu(), inp.k, inp.w, 8, topk_out=topk, workspace=ws)           # no CPU path
    # zero query rows: a no-op
    idxc.indexer_prefill(inp.q[:0], inp.k, inp.w[:0], 8, topk_out=topk[:0], workspace=ws)


# ------------------------------------------------------------------------------ decode
@pytest.mark.parametrize("B,H,d,k_top,fp8,lens,flags", [
    (3, 4, 32, 8, False, [5, 130, 77], idxc.FLAG_SIMT_SCORER),
    (4, 64, 128, 64, False, [1, 127, 1500, 3000], 0),
    (5, 16, 64, 32, False, [129, 2048, 31, 1025, 4000], 0),
    (3, 32, 128, 48, True, [999, 2500, 50], 0),
    (2, 64, 128, 2048, False, [2047, 5000], 0),
    # the remaining (d_I, H_I, dtype) kernels the library accepts
    (3, 32, 64, 16, False, [640, 129, 3000], 0),
    (2, 64, 64, 40, False, [2500, 77], 0),
    (3, 16, 128, 24, False, [128, 1000, 2305], 0),
    (4, 32, 128, 64, False, [1, 2049, 300, 4097], 0),
    (3, 16, 128, 20, True, [700, 2100, 33], 0),
    # FP8 at the paper's head count: several work items per sequence (the key scales are staged one item ahead and the
    # key tiles alternate between two MMA warps), an empty sequence, one of a single key, ragged ends
    (6, 64, 128, 64, True, [0, 9000, 4097, 129, 1, 6500], 0),
    (2, 64, 64, 32, False, [7000, 3333], 0),          # 128-byte rows in bf16: two MMA warps, no scales
])
def test_decode_matches_oracle(B, H, d, k_top, fp8, lens, flags):
    inp = _to_dev(synth.decode_inputs(B, H, d, 0, 0, seed=20 + B, fp8=fp8, lens=lens, row_align=8 if B != 6 else 1))
    ld = (inp.max_len + 3) // 4 * 4
    scores = torch.full((B, ld), float("nan"), device=DEV)
    topk = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.indexer_decode(inp.q_step, inp.k_cache, inp.w, inp.k_offsets, inp.lens, inp.max_len, k_top, inp.q_scale,
                        inp.k_scale, scores_out=scores, topk_out=topk, flags=flags)
    idxc.poll_device_status()
    # without score output (workspace path) the indices are the same
    topk2 = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    ws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, inp.max_len, H, d, k_top), DEV)
    idxc.indexer_decode(inp.q_step, inp.k_cache, inp.w, inp.k_offsets, inp.lens, inp.max_len, k_top, inp.q_scale,
                        inp.k_scale, topk_out=topk2, workspace=ws, flags=flags)
    assert torch.equal(topk, topk2)
    dt = oracle.FP8_E4M3 if fp8 else oracle.BF16
    o_scores, _ = oracle.indexer_decode(codes(inp.q_step), codes(inp.k_cache), f32(inp.w), inp.k_offsets.cpu().numpy(),
                                        inp.lens.cpu().numpy(), k_top, dt, f32(inp.q_scale), f32(inp.k_scale))
    g_scores, g_topk = scores.cpu().numpy(), topk.cpu().numpy()
    rtol = RTOL_FP8 if fp8 else RTOL_BF16
    for b in range(B):
        n = lens[b]
        assert_scores_close(g_scores[b, :n], o_scores[b, :n], rtol, what=f"seq {b}")
        assert np.all(np.isnan(g_scores[b, n:]))
        assert_topk_valid(g_topk[b], o_scores[b, :n], k_top, rtol, what=f"seq {b}")
        order = np.argsort(-g_scores[b, :n].astype(np.float64), kind="stable")
        kk = min(k_top, n)
        assert np.array_equal(np.sort(order[:kk]), g_topk[b, :kk])


def test_decode_equals_prefill_row():
    L, H, d, k_top = 640, 64, 128, 50
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=31))
    s_p, t_p = _gpu_prefill(inp, k_top)
    ts = [0, 127, 128, 300, 639]
    lens = torch.tensor([t + 1 for t in ts], dtype=torch.int32, device=DEV)
    offs = torch.zeros(len(ts), dtype=torch.int64, device=DEV)
    ld = 640
    scores = torch.full((len(ts), ld), float("nan"), device=DEV)
    topk = torch.empty((len(ts), k_top), dtype=torch.int32, device=DEV)
    idxc.indexer_decode(inp.q[ts].contiguous(), inp.k, inp.w[ts].contiguous(), offs, lens, L, k_top,
                        scores_out=scores, topk_out=topk)
    idxc.poll_device_status()
    sc = scores.cpu().numpy()
    for j, t in enumerate(ts):
        assert np.allclose(sc[j, : t + 1], s_p[t, : t + 1], rtol=1e-5, atol=1e-4)   # same products, other tile shape
        o_row = _oracle_prefill(inp, k_top, rows=[t])[0][0, : t + 1]
        assert_topk_valid(topk[j].cpu().numpy(), o_row, k_top, RTOL_BF16)


# ------------------------------------------------------------------------------ schedule
def test_schedule_prefill_shares_bit_for_bit():
    pattern = "FSSFSFSS"
    L, H, d, k_top = 384, 16, 64, 24
    layers = [_to_dev(synth.prefill_inputs(L, H, d, seed=5, layer=l)) for l in range(len(pattern))]
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H, d, k_top), DEV)
    bufs = [torch.full((L, k_top), -9, dtype=torch.int32, device=DEV) for _ in pattern]
    sch = idxc.Schedule(pattern)
    for copy_flag in (0, idxc.FLAG_COPY_SHARED):
        sch.begin_pass()
        before = sch.stats()[2]
        launches0 = idxc.launch_count()
        outs = []
        for l, ch in enumerate(pattern):
            x = layers[l]
            if ch == "F":
                t = sch.prefill_layer(l, x.q, x.k, x.w, k_top, topk_buf=bufs[l], workspace=ws, flags=copy_flag)
            else:   # S layers get no inputs at all: proves they are never read
                t = sch.prefill_layer(l, k_top=k_top, q_len=L, topk_buf=bufs[l] if copy_flag else None, flags=copy_flag)
            outs.append(t)
        idxc.poll_device_status()
        nf, ns, calls = sch.stats()
        assert (nf, ns) == (3, 5) and calls - before == 3
        assert idxc.launch_count() - launches0 == 2 * 3            # scorer + top-k per F layer, nothing on S layers
        src = oracle_schedule.source_layers(pattern)
        for l in range(len(pattern)):
            assert sch.source(l) == src[l]
            assert torch.equal(outs[l], outs[src[l]])
            if copy_flag:
                assert outs[l].data_ptr() == bufs[l].data_ptr()
            else:
                assert outs[l].data_ptr() == bufs[src[l]].data_ptr()   # alias of the F layer's buffer
        # against the oracle's loop, F layers checked with the band criterion
        def oracle_layer(l):
            return _oracle_prefill(layers[l], k_top)[0]
        for l in [0, 3, 5]:
            o_scores = oracle_layer(l)
            g = outs[l].cpu().numpy()
            for t in range(L):
                assert_topk_valid(g[t], o_scores[t, : t + 1], k_top, RTOL_BF16)
    # visiting an S layer before its F layer ran in this pass is an error
    sch.begin_pass()
    with pytest.raises(idxc.IdxcError) as e:
        sch.prefill_layer(1, k_top=k_top, q_len=L)
    assert e.value.status == idxc.ERR_PATTERN
    sch.close()


def test_schedule_decode_layers():
    pattern = "FSFS"
    B, H, d, k_top = 3, 64, 128, 32
    lens = [300, 1000, 129]
    layers = [_to_dev(synth.decode_inputs(B, H, d, 0, 0, seed=8, layer=l, lens=lens)) for l in range(4)]
    sch = idxc.Schedule(pattern)
    sch.begin_pass()
    ws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, 1000, H, d, k_top), DEV)
    bufs = [torch.empty((B, k_top), dtype=torch.int32, device=DEV) for _ in pattern]
    outs = []
    for l, ch in enumerate(pattern):
        x = layers[l]
        if ch == "F":
            outs.append(sch.decode_layer(l, x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top,
                                         topk_buf=bufs[l], workspace=ws))
        else:
            outs.append(sch.decode_layer(l, B=B, k_top=k_top))
    idxc.poll_device_status()
    assert torch.equal(outs[1], outs[0]) and torch.equal(outs[3], outs[2]) and not torch.equal(outs[0], outs[2])
    assert sch.stats() == (2, 2, 2)
    for l in (0, 2):
        x = layers[l]
        o_scores, _ = oracle.indexer_decode(codes(x.q_step), codes(x.k_cache), f32(x.w), x.k_offsets.cpu().numpy(),
                                            x.lens.cpu().numpy(), k_top)
        g = outs[l].cpu().numpy()
        for b in range(B):
            assert_topk_valid(g[b], o_scores[b, : lens[b]], k_top, RTOL_BF16)
    sch.close()


# ------------------------------------------------------------------------------ failure detection
def test_bounded_wait_reports_timeout_and_context_stays_usable():
    """A device-side wait that nothing satisfies runs out (here after ~1e6 cycles), the kernel returns, the
    host reads IDXC_ERR_DEVICE_TIMEOUT once, and the library keeps working afterwards."""
    idxc.poll_device_status()
    idxc.selftest_bounded_wait(1_000_000)
    with pytest.raises(idxc.IdxcError) as e:
        idxc.poll_device_status()
    assert e.value.status == idxc.ERR_DEVICE_TIMEOUT
    idxc.poll_device_status()                               # the record was cleared
    inp = _to_dev(synth.prefill_inputs(256, 16, 64, seed=9))
    g_scores, g_topk = _gpu_prefill(inp, 16)
    _check_prefill(inp, 16, g_scores, g_topk, RTOL_BF16)


# ------------------------------------------------------------------------------ FP8 quantiser (step before the indexer)
@pytest.mark.parametrize("n,shape", [(1, (128,)), (1000, (128,)), (777, (64,)), (300, (256,)), (65, (64, 128)), (33, (16, 64)),
                                    (40, (8, 40)), (5, (8,))])
def test_quantize_e4m3_bit_exact(n, shape):
    g = torch.Generator().manual_seed(n)
    x = (torch.randn((n,) + shape, generator=g) * torch.logspace(-3, 3, n)[(...,) + (None,) * len(shape)]).to(torch.bfloat16)
    if n > 2:
        x[1] = 0                                           # an all-zero token: scale floor, codes 0
    xd = x.to(DEV)
    codes_out = torch.full((n,) + shape, 0x55, dtype=torch.uint8, device=DEV)
    scale_out = torch.full((n,), -1.0, device=DEV)
    idxc.quantize_e4m3(xd, codes_out, scale_out)
    o_codes, o_scale = oracle.quantize_e4m3(codes(x))
    g_codes = codes_out.cpu().numpy()
    assert np.array_equal(scale_out.cpu().numpy(), o_scale)
    nz = (o_codes & 0x7F) != 0
    assert np.array_equal(g_codes & 0x7F, o_codes & 0x7F) and np.array_equal(g_codes[nz], o_codes[nz])


def test_quantize_e4m3_every_value_under_many_row_maxima():
    """The kernel divides by the row's scale through a reciprocal and one residual step instead of a division per
    element. Here rows whose largest entry is a chosen bf16 value hold EVERY bf16 value not above it, both signs: the
    codes must be the oracle's for all of them (edge maxima: subnormal, smallest normal, around the 1e-12 floor, powers
    of two, the largest finite value; plus 200 seeded ones)."""
    g = torch.Generator().manual_seed(5)
    edge = [1, 2, 0x7F, 0x80, 0x81, 0x2B8C, 0x2B8D, 0x2B8E, 0x3F80, 0x3F81, 0x3FFF, 0x4000, 0x43E0, 0x7F00, 0x7F7F]
    maxima = edge + torch.randint(1, 0x7F80, (200,), generator=g).tolist()
    rows = []
    for a in maxima:
        mag = torch.arange(0, a + 1, dtype=torch.int32)
        bits = torch.cat([mag, mag | 0x8000])
        pad = (-bits.numel()) % 127
        bits = torch.cat([bits, torch.zeros(pad, dtype=torch.int32)]).reshape(-1, 127)
        rows.append(torch.cat([torch.full((bits.shape[0], 1), a, dtype=torch.int32), bits], dim=1))
    bits = torch.cat(rows).to(torch.uint16)
    x = bits.view(torch.bfloat16)
    n = x.shape[0]
    codes_out = torch.full((n, 128), 0x55, dtype=torch.uint8, device=DEV)
    scale_out = torch.full((n,), -1.0, device=DEV)
    idxc.quantize_e4m3(x.to(DEV), codes_out, scale_out)
    o_codes, o_scale = oracle.quantize_e4m3(codes(x))
    g_codes = codes_out.cpu().numpy()
    assert np.array_equal(scale_out.cpu().numpy(), o_scale)
    nz = (o_codes & 0x7F) != 0
    assert np.array_equal(g_codes & 0x7F, o_codes & 0x7F) and np.array_equal(g_codes[nz], o_codes[nz])


def test_quantize_e4m3_appends_to_a_k_cache_that_the_indexer_reads():
    # new keys of three sequences are appended at the end of their cache rows, then one decode step reads the cache
    B, H, d, k_top = 3, 64, 128, 32
    lens_before = [200, 511, 64]
    n_new = 1
    base = synth.decode_inputs(B, H, d, 0, 0, seed=50, fp8=True, lens=[l + n_new for l in lens_before], row_align=128)
    base = _to_dev(base)
    g = torch.Generator().manual_seed(51)
    new_keys = torch.randn(B, d, generator=g).to(torch.bfloat16).to(DEV)
    dst = (base.k_offsets + torch.tensor(lens_before, device=DEV)).to(torch.int64)
    idxc.quantize_e4m3(new_keys, base.k_cache.view(torch.uint8), base.k_scale, dst_rows=dst)
    o_codes, o_scale = oracle.quantize_e4m3(codes(new_keys))
    kc = base.k_cache.view(torch.uint8).cpu().numpy()
    for b in range(B):
        row = int(dst[b])
        assert np.array_equal(kc[row] & 0x7F, o_codes[b] & 0x7F)
        assert base.k_scale[row].item() == o_scale[b]
    topk = torch.empty((B, k_top), dtype=torch.int32, device=DEV)
    ws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, base.max_len, H, d, k_top, idxc.FP8_E4M3), DEV)
    idxc.indexer_decode(base.q_step, base.k_cache, base.w, base.k_offsets, base.lens, base.max_len, k_top, base.q_scale,
                        base.k_scale, topk_out=topk, workspace=ws)
    idxc.poll_device_status()
    o_sc, _ = oracle.indexer_decode(codes(base.q_step), codes(base.k_cache), f32(base.w), base.k_offsets.cpu().numpy(),
                                    base.lens.cpu().numpy(), k_top, oracle.FP8_E4M3, f32(base.q_scale), f32(base.k_scale))
    for b in range(B):
        assert_topk_valid(topk[b].cpu().numpy(), o_sc[b, : lens_before[b] + n_new], k_top, RTOL_FP8)


# ------------------------------------------------------------------------------ pattern tooling: top-k overlap (Appendix A)
def test_topk_overlap_matches_oracle():
    from oracle import pattern as opat
    L, H, d, k_top = 700, 16, 64, 64
    n_layers = 4
    tops = []
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H, d, k_top), DEV)
    for l in range(n_layers):
        inp = synth.prefill_inputs(L, H, d, seed=60, layer=l // 2)       # layers 0,1 and 2,3 share inputs
        if l % 2 == 1:
            inp.w = inp.w * (1.0 + 0.5 * torch.randn(inp.w.shape, generator=torch.Generator().manual_seed(l)))
        inp = _to_dev(inp)
        t = torch.empty((L, k_top), dtype=torch.int32, device=DEV)
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, topk_out=t, workspace=ws)
        tops.append(t)
    mean = idxc.topk_overlap(tops).cpu().numpy()
    pairs = [(a, b) for a in range(n_layers) for b in range(a + 1, n_layers)]
    host = [t.cpu().numpy() for t in tops]
    for p, (a, b) in enumerate(pairs):
        assert mean[p] == pytest.approx(opat.overlap(host[a], host[b]), abs=1e-9)
    m1, rows = idxc.topk_overlap(tops, pairs=[(1, 0)], want_rows=True)
    assert np.allclose(rows.cpu().numpy(), opat.overlap_rows(host[1], host[0]), atol=1e-6)
    assert idxc.topk_overlap([tops[0], tops[0]]).item() == 1.0          # identical tensors overlap fully


@pytest.mark.parametrize("k_top,max_index", [(2048, 16384), (2048, 131072), (2048, 400000), (37, 5000), (37, 300000), (512, 131073)])
def test_topk_overlap_near_and_far_rows_mixed(k_top, max_index):
    """Rows whose largest index is below 131072 are intersected through a bitmap, the others by merging; here both kinds
    alternate inside one launch (so a merged row must leave the bitmap clean), with padded, empty and identical rows."""
    from oracle import pattern as opat
    rows = 97
    g = torch.Generator().manual_seed(k_top + max_index)

    def tensor(shift):
        t = torch.full((rows, k_top), -1, dtype=torch.int32)
        for r in range(rows):
            hi = max_index if r % 3 else min(max_index, 9000)             # every third row stays near
            n = k_top if r % 5 else int(torch.randint(0, k_top + 1, (1,), generator=g))
            n = min(n, hi)
            if r == 11:
                n = 0                                                     # an empty row
            pick = torch.randperm(hi, generator=g)[:n]
            if shift and r % 2:
                pick = torch.cat([pick[: n // 2], torch.randperm(hi, generator=g)[: n - n // 2]]).unique()
            vals = torch.sort(pick.unique()).values
            t[r, : vals.numel()] = vals.to(torch.int32)
        return t
    a, b = tensor(False), tensor(True)
    b[20] = a[20]                                                         # an identical row
    tops = [a.to(DEV), b.to(DEV)]
    for pair, (x, y) in (((0, 1), (a, b)), ((1, 0), (b, a))):
        mean, per_row = idxc.topk_overlap(tops, pairs=[pair], want_rows=True)
        want = opat.overlap_rows(x.numpy(), y.numpy())
        assert np.allclose(per_row.cpu().numpy(), want, atol=1e-6)
        assert mean.item() == pytest.approx(float(np.mean(want)), abs=1e-9)
    both = idxc.topk_overlap(tops, pairs=[(0, 1), (1, 0), (0, 0)]).cpu().numpy()
    assert both[0] == pytest.approx(opat.overlap(a.numpy(), b.numpy()), abs=1e-9)
    assert both[1] == pytest.approx(opat.overlap(b.numpy(), a.numpy()), abs=1e-9)
    assert both[2] == pytest.approx(opat.overlap(a.numpy(), a.numpy()), abs=1e-9)


# ------------------------------------------------------------------------------ multi-layer distillation loss (Eq. 1)
def test_distill_kl_matches_oracle():
    from oracle import distill as odist
    L, H, d, k_top = 300, 16, 64, 32
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=70))
    g_scores, g_topk = _gpu_prefill(inp, k_top)
    scores = torch.nan_to_num(torch.from_numpy(g_scores), nan=0.0).to(DEV).contiguous()      # entries above the diagonal are unused
    gen = torch.Generator().manual_seed(71)
    targets = []
    for j in range(3):
        p = torch.rand((L, scores.shape[1]), generator=gen) * torch.tril(torch.ones(L, scores.shape[1]))
        p[:, 5] = 0.0                                           # exact zeros in a target contribute nothing
        p[5, 5] = 1.0
        targets.append((p / p.sum(dim=1, keepdim=True)).to(DEV).contiguous())
    loss, rows = idxc.distill_kl(scores, targets, want_rows=True)
    want, want_rows = odist.multi_layer_loss(scores.cpu().numpy(), [t.cpu().numpy() for t in targets])
    assert loss.item() == pytest.approx(want, rel=2e-5)
    assert np.allclose(rows.cpu().numpy(), want_rows, rtol=1e-4, atol=1e-6)
    # more targets than one sweep holds in registers (groups of four), and a single one
    more = targets + [targets[0].flip(0).contiguous() * 0 + targets[1], targets[2], targets[0]]
    for tl in (more, targets[:1]):
        loss_m, rows_m = idxc.distill_kl(scores, tl, want_rows=True)
        want_m, want_rows_m = odist.multi_layer_loss(scores.cpu().numpy(), [t.cpu().numpy() for t in tl])
        assert loss_m.item() == pytest.approx(want_m, rel=2e-5)
        assert np.allclose(rows_m.cpu().numpy(), want_rows_m, rtol=1e-4, atol=1e-6)
    # sparse-training form on the indices the top-k kernel selected
    tk = torch.from_numpy(g_topk).to(DEV)
    loss_k, rows_k = idxc.distill_kl(scores, targets, topk=tk, want_rows=True)
    want_k, want_rows_k = odist.multi_layer_loss(scores.cpu().numpy(), [t.cpu().numpy() for t in targets], topk=g_topk)
    assert loss_k.item() == pytest.approx(want_k, rel=2e-5)
    assert np.allclose(rows_k.cpu().numpy(), want_rows_k, rtol=1e-4, atol=1e-6)
    # the loss of the Softmax of the scores against itself is zero
    q = torch.softmax(scores.masked_fill(torch.triu(torch.ones_like(scores, dtype=torch.bool), diagonal=1), float("-inf")), dim=1)
    assert abs(idxc.distill_kl(scores, [q.contiguous()]).item()) < 1e-3 * L
