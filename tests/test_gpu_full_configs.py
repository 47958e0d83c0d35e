"""Parity at the full sizes of the five workloads, in the launch configuration bench.py times.
The oracle is evaluated on a deterministic sample of whole rows (edges, tile and chunk borders,
a few seeded random rows); properties that hold at any size (row length, order, range, padding,
Shared == Full) are checked over the whole GPU output."""
import numpy as np
import pytest
import torch

import oracle
from paper_2603_12201_b200 import binding as idxc
from paper_2603_12201_b200 import synth
from tests.util import RTOL_BF16, RTOL_FP8, assert_scores_close, assert_topk_valid, codes, f32

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _structure_ok(topk: torch.Tensor, q_begin: int, k_top: int):
    """Whole-output structural check on the device: per row min(k, t+1) strictly ascending indices in
    [0, t], then -1 padding."""
    rows = topk.shape[0]
    t = torch.arange(q_begin, q_begin + rows, device=topk.device)
    kk = torch.clamp(t + 1, max=k_top)
    col = torch.arange(k_top, device=topk.device)
    valid = col[None, :] < kk[:, None]
    assert bool(((topk >= 0) == valid).all()), "count / padding"
    assert bool((torch.where(valid, topk.long(), torch.zeros_like(topk, dtype=torch.long)) <= t[:, None]).all()), "causality"
    d = topk[:, 1:] - topk[:, :-1]
    assert bool((d[valid[:, 1:]] > 0).all()), "strictly ascending"
    assert bool((topk[~valid] == -1).all())


def _sample_rows(L, k_top, extra_seed, n_random=6, chunk=None):
    rows = {0, 1, k_top - 1, k_top, k_top + 1, 127, 128, 129, L // 2, L - 2, L - 1}
    if chunk:
        rows |= {chunk - 1, chunk, L - chunk, L - chunk - 1}
    rng = np.random.default_rng(extra_seed)
    rows |= set(int(x) for x in rng.integers(k_top, L, size=n_random))
    return sorted(r for r in rows if 0 <= r < L)


def _check_sampled(inp, k_top, topk_dev, rows, rtol, score_rows=None):
    """Oracle on the sampled rows (each row evaluated at its own position)."""
    dt = oracle.FP8_E4M3 if inp.fp8 else oracle.BF16
    exact = 0
    for t in rows:
        q1 = codes(inp.q[t:t + 1])
        w1 = f32(inp.w[t:t + 1])
        qs1 = None if inp.q_scale is None else f32(inp.q_scale[t:t + 1])
        o_sc, _ = oracle.indexer_prefill(q1, codes_cached(inp), w1, k_top, dt, qs1, f32(inp.k_scale), q_begin=t)
        o_row = o_sc[0, : t + 1]
        exact += assert_topk_valid(topk_dev[t].cpu().numpy(), o_row, k_top, rtol, what=f"row {t}")
        if score_rows is not None and t in score_rows:
            assert_scores_close(score_rows[t][: t + 1], o_row, rtol, what=f"row {t}")
    return exact / len(rows)


_codes_cache = {}


def codes_cached(inp):
    """Host copy of the current inputs' key codes, made once per input set. The cache keeps the tensor itself and compares
    by identity: an `id()` alone can come back for a new tensor once the old one has been freed."""
    if _codes_cache.get("k") is not inp.k:
        _codes_cache["k"] = inp.k
        _codes_cache["codes"] = codes(inp.k)
    return _codes_cache["codes"]


def _gpu_row_scores(inp, t, k_top):
    """Scores of one row through a one-row chunked call (q_begin = t)."""
    L = inp.k.shape[0]
    sc = torch.full((1, L), float("nan"), device=DEV)
    qs = None if inp.q_scale is None else inp.q_scale[t:t + 1].contiguous()
    idxc.indexer_prefill(inp.q[t:t + 1].contiguous(), inp.k, inp.w[t:t + 1].contiguous(), k_top, qs, inp.k_scale,
                         q_begin=t, scores_out=sc)
    return sc[0].cpu().numpy()


def test_config2_full_size_sampled_rows():
    c = synth.CONFIGS["cfg2"]
    L, H, d, k_top = c["L"], c["H"], c["d"], c["k_top"]
    inp = synth.prefill_inputs(L, H, d, seed=c["seed"], device=DEV, clustered=True)
    topk = torch.full((L, k_top), -7, dtype=torch.int32, device=DEV)
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H, d, k_top), DEV)
    idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, topk_out=topk, workspace=ws)
    idxc.poll_device_status()
    _structure_ok(topk, 0, k_top)
    rows = _sample_rows(L, k_top, extra_seed=2)
    score_rows = {t: _gpu_row_scores(inp, t, k_top) for t in rows[::3]}
    frac = _check_sampled(inp, k_top, topk, rows, RTOL_BF16, score_rows)
    assert frac >= 0.9


def test_config3_full_size_decode_sampled_sequences():
    c = synth.CONFIGS["cfg3"]
    B, H, d, k_top = c["B"], c["H"], c["d"], c["k_top"]
    x = synth.decode_inputs(B, H, d, c["len_lo"], c["len_hi"], seed=c["seed"], device=DEV)
    topk = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    ws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, x.max_len, H, d, k_top), DEV)
    idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, topk_out=topk, workspace=ws)
    topk_na = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.indexer_decode_noalloc(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, topk_na)
    idxc.poll_device_status()
    assert torch.equal(topk, topk_na)
    lens = x.lens.cpu().numpy()
    assert lens.min() >= c["len_lo"] and lens.max() <= c["len_hi"]
    g = topk.cpu().numpy()
    for b in range(B):                                   # structure of every sequence
        assert np.all(np.diff(g[b]) > 0) and g[b, 0] >= 0 and g[b, -1] < lens[b]
    picks = sorted({int(np.argmin(lens)), int(np.argmax(lens)), 3, 17})
    sub = torch.tensor(picks)
    o_sc, _ = oracle.indexer_decode(codes(x.q_step[sub]), codes(x.k_cache), f32(x.w[sub]), x.k_offsets[sub].cpu().numpy(),
                                    lens[picks], k_top)
    for j, b in enumerate(picks):
        assert_topk_valid(g[b], o_sc[j, : lens[b]], k_top, RTOL_BF16, what=f"seq {b}")


def test_config4_shape_schedule_reduced_layers():
    c = synth.CONFIGS["cfg4"]
    L, H, d, k_top = c["L"], c["H"], c["d"], c["k_top"]
    n_layers = 8                                          # the workload has 48; 8 keep the test in seconds
    pattern = synth.uniform_pattern(n_layers, c["every"])
    assert pattern == "FSSSFSSS"
    sch = idxc.Schedule(pattern)
    sch.begin_pass()
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H, d, k_top), DEV)
    outs, full_inputs = [], {}
    for l, ch in enumerate(pattern):
        if ch == "F":
            inp = synth.prefill_inputs(L, H, d, seed=c["seed"], device=DEV, layer=l)
            buf = torch.full((L, k_top), -7, dtype=torch.int32, device=DEV)
            outs.append(sch.prefill_layer(l, inp.q, inp.k, inp.w, k_top, topk_buf=buf, workspace=ws))
            full_inputs[l] = inp
        else:
            outs.append(sch.prefill_layer(l, k_top=k_top, q_len=L))
    idxc.poll_device_status()
    assert sch.stats() == (2, 6, 2)
    for l in range(n_layers):
        src = sch.source(l)
        assert outs[l].data_ptr() == outs[src].data_ptr()
    assert not torch.equal(outs[0], outs[4])
    for l in (0, 4):
        _structure_ok(outs[l], 0, k_top)
        rows = _sample_rows(L, k_top, extra_seed=10 + l, n_random=3)
        _check_sampled(full_inputs[l], k_top, outs[l], rows, RTOL_BF16)
    sch.close()


def test_config5_fp8_chunked_prefill_and_decode():
    c = synth.CONFIGS["cfg5"]
    L, H, d, k_top, chunk = c["L"], c["H"], c["d"], c["k_top"], c["chunk"]
    inp = synth.prefill_inputs(L, H, d, seed=c["seed"], device=DEV, fp8=True)
    topk = torch.full((L, k_top), -7, dtype=torch.int32, device=DEV)
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(chunk, L, H, d, k_top, idxc.FP8_E4M3), DEV)
    for q0 in range(0, L, chunk):                          # 16 chunks of 8192 query rows against the full causal K
        sl = slice(q0, q0 + chunk)
        idxc.indexer_prefill(inp.q[sl], inp.k, inp.w[sl], k_top, inp.q_scale[sl], inp.k_scale, q_begin=q0,
                             topk_out=topk[sl], workspace=ws)
    idxc.poll_device_status()
    _structure_ok(topk, 0, k_top)
    rows = _sample_rows(L, k_top, extra_seed=5, n_random=4, chunk=chunk)
    score_rows = {t: _gpu_row_scores(inp, t, k_top) for t in (rows[3], rows[-1])}
    _check_sampled(inp, k_top, topk, rows, RTOL_FP8, score_rows)
    # the GPU scores on the same FP8 bytes are in fact far inside the bf16-grade bound
    t = rows[-1]
    dt = oracle.FP8_E4M3
    o_sc, _ = oracle.indexer_prefill(codes(inp.q[t:t + 1]), codes_cached(inp), f32(inp.w[t:t + 1]), k_top, dt,
                                     f32(inp.q_scale[t:t + 1]), f32(inp.k_scale), q_begin=t)
    assert_scores_close(score_rows[t][: t + 1], o_sc[0, : t + 1], RTOL_BF16, what="fp8 row, tight bound")
    # the streaming top-k on the first, a middle and the last chunk: the same indices entry for entry. The last chunk's rows
    # are so long that the sample leaves the threshold loose, most of its work items overflow a list and are scored again by
    # the ordinary kernels: the path that repairs is exercised at scale
    F = idxc.FLAG_STREAM_TOPK
    ws_s = idxc.alloc_workspace(idxc.prefill_workspace_bytes(chunk, L, H, d, k_top, idxc.FP8_E4M3, F), DEV)
    for q0 in (0, 7 * chunk, L - chunk):
        sl = slice(q0, q0 + chunk)
        t_s = torch.full((chunk, k_top), -7, dtype=torch.int32, device=DEV)
        idxc.indexer_prefill(inp.q[sl], inp.k, inp.w[sl], k_top, inp.q_scale[sl], inp.k_scale, q_begin=q0, topk_out=t_s,
                             workspace=ws_s, flags=F)
        idxc.poll_device_status()
        assert torch.equal(t_s, topk[sl]), f"streaming top-k, chunk at {q0}"
    del ws_s
    # one decode step at the workload's batch: the resulting cache (sequence 0) and fresh caches of the same length
    B = c["decode_B"]
    fresh = synth.decode_inputs(B, H, d, L, L, seed=c["seed"], device=DEV, layer=1, fp8=True, lens=[L] * B)
    fresh.k_cache[:L] = inp.k
    fresh.k_scale[:L] = inp.k_scale
    d_topk = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    dws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, L, H, d, k_top, idxc.FP8_E4M3), DEV)
    idxc.indexer_decode(fresh.q_step, fresh.k_cache, fresh.w, fresh.k_offsets, fresh.lens, L, k_top, fresh.q_scale,
                        fresh.k_scale, topk_out=d_topk, workspace=dws)
    idxc.poll_device_status()
    o_sc, _ = oracle.indexer_decode(codes(fresh.q_step), codes(fresh.k_cache), f32(fresh.w), fresh.k_offsets.cpu().numpy(),
                                    fresh.lens.cpu().numpy(), k_top, dt, f32(fresh.q_scale), f32(fresh.k_scale))
    g = d_topk.cpu().numpy()
    for b in range(B):
        assert_topk_valid(g[b], o_sc[b, :L], k_top, RTOL_FP8, what=f"decode seq {b}")
