"""GPU parity of the streaming top-k (IDXC_FLAG_STREAM_TOPK): the prefill scorer keeps per query row only the scores
that can still be among the k_top largest, a second kernel selects exactly from those lists, and rows whose list cannot
give the answer go through the ordinary score + select kernels. The indices must be those of the ordinary path entry for
entry, and valid against the FP64 oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_12201_b200 import binding as idxc
from paper_2603_12201_b200 import synth
from tests.util import RTOL_BF16, RTOL_FP8, assert_topk_valid, codes, f32

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _to_dev(inp):
    for name in ("q", "k", "w", "q_scale", "k_scale"):
        if getattr(inp, name, None) is not None:
            setattr(inp, name, getattr(inp, name).to(DEV))
    return inp


def _dtype(inp):
    return idxc.FP8_E4M3 if inp.fp8 else idxc.BF16


def _run(inp, k_top, stream, q_begin=0, q_slice=None, workspace=None):
    q, w, qs = inp.q, inp.w, inp.q_scale
    if q_slice is not None:
        q, w = q[q_slice].contiguous(), w[q_slice].contiguous()
        qs = None if qs is None else qs[q_slice].contiguous()
    q_len, L_k = q.shape[0], inp.k.shape[0]
    flags = idxc.FLAG_STREAM_TOPK if stream else 0
    topk = torch.full((q_len, k_top), -7, dtype=torch.int32, device=DEV)
    if workspace is None:
        workspace = idxc.alloc_workspace(idxc.prefill_workspace_bytes(q_len, L_k, q.shape[1], q.shape[2], k_top, _dtype(inp), flags), DEV)
    before = idxc.launch_count()
    idxc.indexer_prefill(q, inp.k, w, k_top, qs, inp.k_scale, q_begin=q_begin, topk_out=topk, workspace=workspace, flags=flags)
    idxc.poll_device_status()
    return topk.cpu().numpy(), idxc.launch_count() - before


@pytest.mark.parametrize("L,H,d,k_top,fp8", [
    (3000, 64, 128, 256, False),        # several work items, ragged last key tile, a sample stride of 3
    (5000, 64, 128, 2048, False),       # k_top at its maximum: rows up to 2048 keys keep everything
    (2500, 32, 64, 64, False),          # 16 rows per work item, 4 sample tiles
    (2100, 16, 128, 100, True),         # 32 rows per work item, 2 sample tiles, e4m3 with scales
    (4200, 64, 128, 512, True),
    (900, 64, 128, 1024, False),        # every row shorter than k_top: no threshold anywhere
    (1, 64, 128, 4, False),
])
def test_stream_topk_equals_the_ordinary_path_and_the_oracle(L, H, d, k_top, fp8):
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=300 + L, fp8=fp8))
    t_ord, n_ord = _run(inp, k_top, stream=False)
    t_str, n_str = _run(inp, k_top, stream=True)
    assert n_ord == 2 and n_str == 4              # scorer + select; scorer, list select, and the two kernels for flagged rows
    assert np.array_equal(t_str, t_ord)
    rows = sorted(set([0, 1, L // 3, L // 2, L - 2, L - 1]) & set(range(L)))
    dt = oracle.FP8_E4M3 if fp8 else oracle.BF16
    o_scores, _ = oracle.indexer_prefill(codes(inp.q), codes(inp.k), f32(inp.w), k_top, dt, f32(inp.q_scale), f32(inp.k_scale), rows=rows)
    for j, t in enumerate(rows):
        assert_topk_valid(t_str[t], o_scores[j, : t + 1], k_top, RTOL_FP8 if fp8 else RTOL_BF16, what=f"row {t}")


def test_stream_topk_chunks_of_queries_and_of_the_workspace():
    L, H, d, k_top = 2600, 64, 128, 128
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=41))
    t_ord, _ = _run(inp, k_top, stream=False)
    # query chunks against the full K
    for q0, q1 in [(0, 500), (500, 1700), (1700, 2600)]:
        t_c, _ = _run(inp, k_top, stream=True, q_begin=q0, q_slice=slice(q0, q1))
        assert np.array_equal(t_c, t_ord[q0:q1])
    # a workspace for 64 rows at a time: 41 chunks, four launches each
    per_row = idxc.prefill_workspace_bytes(64, L, H, d, k_top, idxc.BF16, idxc.FLAG_STREAM_TOPK)
    t_small, n = _run(inp, k_top, stream=True, workspace=idxc.alloc_workspace(per_row, DEV))
    assert np.array_equal(t_small, t_ord)
    assert n == 4 * ((L + 63) // 64)
    with pytest.raises(idxc.IdxcError) as e:
        _run(inp, k_top, stream=True, workspace=idxc.alloc_workspace(per_row // 8, DEV))
    assert e.value.status == idxc.ERR_WORKSPACE


def test_stream_topk_rows_the_lists_cannot_answer_take_the_ordinary_path():
    """Equal scores in bulk: with w = 0 every score of a row is 0, no threshold separates them, the per-thread lists of
    long rows overflow and short rows have more equal scores at the threshold than the list select ranks. Both kinds
    must come out as the lowest positions, from the ordinary kernels. Rows of a second kind: all scores distinct but
    growing with the key position, so that the k_top largest are the last ones."""
    L, H, d, k_top = 12000, 64, 128, 300
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=5))
    inp.w.zero_()
    t_str, _ = _run(inp, k_top, stream=True)
    for t in (0, 299, 300, 5000, 8200, 8500, L - 1):
        kk = min(k_top, t + 1)
        assert np.array_equal(t_str[t, :kk], np.arange(kk)), f"row {t}"
        assert np.all(t_str[t, kk:] == -1)
    # the same through a workspace of 96 rows: the flags of a chunk's rows and work items are the chunk's own
    small = idxc.alloc_workspace(idxc.prefill_workspace_bytes(96, L, H, d, k_top, idxc.BF16, idxc.FLAG_STREAM_TOPK), DEV)
    t_small, _ = _run(inp, k_top, stream=True, workspace=small)
    assert np.array_equal(t_small, t_str)
    # scores that grow with the position: q = k = e_0 scaled by the position, one head with weight 1
    L = 6000
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=6))
    inp.q.zero_(); inp.k.zero_(); inp.w.zero_()
    inp.q[:, 0, 0] = 1.0
    inp.w[:, 0] = 1.0
    inp.k[:, 0] = (torch.arange(L, device=DEV, dtype=torch.float32) / 64.0 + 1.0).to(inp.k.dtype)   # bf16: runs of equal values
    t_ord, _ = _run(inp, k_top, stream=False)
    t_str, _ = _run(inp, k_top, stream=True)
    assert np.array_equal(t_str, t_ord)


def test_stream_topk_argument_checks():
    L, H, d, k_top = 256, 64, 128, 16
    inp = _to_dev(synth.prefill_inputs(L, H, d, seed=2))
    topk = torch.empty((L, k_top), dtype=torch.int32, device=DEV)
    scores = torch.empty((L, L), dtype=torch.float32, device=DEV)
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H, d, k_top, idxc.BF16, idxc.FLAG_STREAM_TOPK), DEV)
    with pytest.raises(idxc.IdxcError) as e:          # the streaming form writes no scores
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, scores_out=scores, topk_out=topk, workspace=ws, flags=idxc.FLAG_STREAM_TOPK)
    assert e.value.status == idxc.ERR_INVALID_ARG
    with pytest.raises(idxc.IdxcError) as e:          # not with the CUDA-core scorer
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, topk_out=topk, workspace=ws, flags=idxc.FLAG_STREAM_TOPK | idxc.FLAG_SIMT_SCORER)
    assert e.value.status == idxc.ERR_INVALID_ARG
    with pytest.raises(idxc.IdxcError) as e:          # no workspace
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, topk_out=topk, flags=idxc.FLAG_STREAM_TOPK)
    assert e.value.status == idxc.ERR_WORKSPACE
