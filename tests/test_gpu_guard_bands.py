"""Out-of-bounds writes and run-to-run determinism of every kernel, without a memory checker.

Every output and workspace buffer of a call is carved out of a larger allocation with a sentinel-filled band in
front of it and behind it; after the call the bands must still hold the sentinel (a kernel that writes one row past
its output, one column past a row pitch or beyond its workspace share would change them). Each call is then repeated
on the same inputs and must reproduce its outputs bit for bit, which catches most races between the roles of a
kernel. Sizes are odd on purpose (ragged tiles, partial work items, row pitches larger than the rows).
"""
import numpy as np
import pytest
import torch

from paper_2603_12201_b200 import binding as idxc
from paper_2603_12201_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
BAND = 8192          # bytes in front of and behind every guarded buffer (a multiple of the 256-byte workspace alignment)
SENTINEL = 0xA5


class Guarded:
    """A tensor of `shape`/`dtype` with sentinel bands around it; `fill` initialises the payload."""

    def __init__(self, shape, dtype, fill=None):
        n = int(np.prod(shape)) * torch.empty((), dtype=dtype).element_size()
        self.nbytes = n
        self.raw = torch.full((BAND + (n + 255) // 256 * 256 + BAND,), SENTINEL, dtype=torch.uint8, device=DEV)
        self.t = self.raw[BAND:BAND + n].view(dtype).view(shape)
        if fill is not None:
            self.t.fill_(fill)

    def check(self, what):
        head = self.raw[:BAND]
        tail = self.raw[BAND + self.nbytes:]
        assert bool((head == SENTINEL).all()), f"{what}: bytes in front of the buffer were written"
        assert bool((tail == SENTINEL).all()), f"{what}: bytes behind the buffer were written"


def _twice(run, outputs, what):
    """Runs `run()` twice; `outputs` lists Guarded buffers whose payload must agree bit for bit between the runs and whose
    bands must be intact after each."""
    initial = [g.t.clone() for g in outputs]
    run()
    idxc.poll_device_status()
    first = [g.t.clone() for g in outputs]
    for g in outputs:
        g.check(what)
    for g, init in zip(outputs, initial):               # back to the initial fill, so that a skipped write shows
        g.t.copy_(init)
    run()
    idxc.poll_device_status()
    for g, f in zip(outputs, first):
        g.check(what + " (second run)")
        assert torch.equal(g.t.view(torch.uint8), f.view(torch.uint8)), f"{what}: second run differs"


def _dev(inp):
    for name in ("q", "k", "w", "q_scale", "k_scale", "q_step", "k_cache", "k_offsets", "lens"):
        if hasattr(inp, name) and getattr(inp, name) is not None:
            setattr(inp, name, getattr(inp, name).to(DEV))
    return inp


@pytest.mark.parametrize("L,H,d,k_top,fp8", [(1, 64, 128, 8, False), (127, 64, 128, 40, False), (129, 16, 64, 16, False),
                                              (2049, 64, 128, 300, False), (777, 32, 128, 64, True), (515, 64, 128, 2048, True)])
def test_prefill_outputs_and_workspace(L, H, d, k_top, fp8):
    inp = _dev(synth.prefill_inputs(L, H, d, seed=1000 + L, fp8=fp8))
    ld = (L + 3) // 4 * 4 + 8                                       # pitch wider than the row: columns >= L must stay untouched
    # (a) scores and indices to caller buffers; the score payload starts as the sentinel so the entries s > t can be checked too
    scores = Guarded((L, ld), torch.float32)
    topk = Guarded((L, k_top), torch.int32)

    def run_a():
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, inp.q_scale, inp.k_scale, scores_out=scores.t, topk_out=topk.t)
    run_a()
    idxc.poll_device_status()
    scores.check("prefill scores")
    topk.check("prefill indices")
    raw = scores.t.view(torch.int32)
    t = torch.arange(L, device=DEV)[:, None]
    s_ = torch.arange(ld, device=DEV)[None, :]
    untouched = raw[(s_ > t).expand(L, ld)]
    assert bool((untouched == int.from_bytes(bytes([SENTINEL] * 4), "little", signed=True)).all()), "entries s > t were written"
    ref_scores, ref_topk = scores.t.clone(), topk.t.clone()
    run_a()
    idxc.poll_device_status()
    assert torch.equal(scores.t.view(torch.int32), ref_scores.view(torch.int32)) and torch.equal(topk.t, ref_topk)
    # (b) scores through a guarded workspace, whole and in several chunks
    dt = idxc.FP8_E4M3 if fp8 else idxc.BF16
    full = idxc.prefill_workspace_bytes(L, L, H, d, k_top, dt)
    small = idxc.prefill_workspace_bytes(64, L, H, d, k_top, dt)    # room for 64 rows at a time: several chunks
    for nbytes in sorted({full, min(full, small)}):
        ws = Guarded((max(nbytes, 256),), torch.uint8)
        top2 = Guarded((L, k_top), torch.int32, fill=-7)
        _twice(lambda: idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, inp.q_scale, inp.k_scale, topk_out=top2.t, workspace=ws.t),
               [top2], f"prefill through a {nbytes}-byte workspace")
        ws.check("prefill workspace")
        assert torch.equal(top2.t, ref_topk)
    # (c) a query chunk against the full K
    if L > 64:
        q0, q1 = L // 3, L - 5
        part = Guarded((q1 - q0, k_top), torch.int32, fill=-7)
        ws = Guarded((idxc.prefill_workspace_bytes(q1 - q0, L, H, d, k_top, dt),), torch.uint8)
        qs = None if inp.q_scale is None else inp.q_scale[q0:q1].contiguous()
        _twice(lambda: idxc.indexer_prefill(inp.q[q0:q1].contiguous(), inp.k, inp.w[q0:q1].contiguous(), k_top, qs, inp.k_scale,
                                            q_begin=q0, topk_out=part.t, workspace=ws.t), [part], "chunked prefill")
        ws.check("chunk workspace")
        assert torch.equal(part.t, ref_topk[q0:q1])


@pytest.mark.parametrize("L,H,d,k_top,fp8,rows_ws", [(2049, 64, 128, 300, False, 0), (1300, 64, 128, 2048, True, 64), (777, 32, 64, 64, False, 0),
                                                      (515, 16, 128, 40, True, 32)])
def test_streaming_topk_outputs_and_workspace(L, H, d, k_top, fp8, rows_ws):
    """The streaming top-k writes per-row candidate lists, list lengths, thresholds and flag bytes into regions of the
    workspace: nothing of it may land outside the workspace or the index output, whole or in chunks of rows_ws rows."""
    inp = _dev(synth.prefill_inputs(L, H, d, seed=2000 + L, fp8=fp8))
    dt = idxc.FP8_E4M3 if fp8 else idxc.BF16
    F = idxc.FLAG_STREAM_TOPK
    topk = Guarded((L, k_top), torch.int32, fill=-7)
    ws = Guarded((idxc.prefill_workspace_bytes(rows_ws or L, L, H, d, k_top, dt, F),), torch.uint8)

    def run():
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, inp.q_scale, inp.k_scale, topk_out=topk.t, workspace=ws.t, flags=F)
    _twice(run, [topk], "streaming prefill")
    ws.check("streaming prefill workspace")
    # and it is the ordinary path's answer
    ref = torch.empty((L, k_top), dtype=torch.int32, device=DEV)
    idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, inp.q_scale, inp.k_scale, topk_out=ref,
                         workspace=idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H, d, k_top, dt), DEV))
    assert torch.equal(ref, topk.t)


@pytest.mark.parametrize("H,d,k_top,fp8,lens", [(64, 128, 64, False, [1, 127, 129, 2049]), (16, 64, 16, False, [300, 5, 4097]),
                                                 (64, 128, 2048, True, [2047, 2049, 9000]), (32, 128, 100, True, [515])])
def test_decode_outputs_workspace_and_builtin_scratch(H, d, k_top, fp8, lens):
    B = len(lens)
    x = _dev(synth.decode_inputs(B, H, d, 0, 0, seed=2000 + B, fp8=fp8, lens=lens, row_align=8))
    ld = (x.max_len + 3) // 4 * 4 + 4
    scores = Guarded((B, ld), torch.float32, fill=float("nan"))
    topk = Guarded((B, k_top), torch.int32, fill=-7)
    _twice(lambda: idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, x.q_scale, x.k_scale,
                                       scores_out=scores.t, topk_out=topk.t), [scores, topk], "decode to caller buffers")
    for b in range(B):
        assert bool(torch.isnan(scores.t[b, lens[b]:]).all()), "scores beyond the sequence length were written"
    dt = idxc.FP8_E4M3 if fp8 else idxc.BF16
    ws = Guarded((idxc.decode_workspace_bytes(B, x.max_len, H, d, k_top, dt),), torch.uint8)
    top2 = Guarded((B, k_top), torch.int32, fill=-7)
    _twice(lambda: idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, x.q_scale, x.k_scale,
                                       topk_out=top2.t, workspace=ws.t), [top2], "decode through the workspace")
    ws.check("decode workspace")
    top3 = Guarded((B, k_top), torch.int32, fill=-7)
    _twice(lambda: idxc.indexer_decode_noalloc(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, top3.t,
                                               x.q_scale, x.k_scale), [top3], "decode with the built-in scratch")
    assert torch.equal(top2.t, topk.t) and torch.equal(top3.t, topk.t)


@pytest.mark.parametrize("n_rows,ld,k_top", [(3, 20000, 2048), (1100, 1300, 256), (70, 132, 16), (9, 70000, 500)])
def test_topk_alone(n_rows, ld, k_top):
    g = torch.Generator().manual_seed(n_rows)
    s = torch.randn(n_rows, ld, generator=g)
    s[0] = 0.0
    lens = torch.randint(1, ld + 1, (n_rows,), generator=g, dtype=torch.int32)
    lens[-1] = ld
    sd, ld_ = s.to(DEV), lens.to(DEV)
    out = Guarded((n_rows, k_top), torch.int32, fill=-7)
    _twice(lambda: idxc.topk_rows(sd, k_top, out.t, lens=ld_), [out], "top-k")


def test_quantiser_with_and_without_row_scatter():
    for n, row in ((1, 8), (777, 64), (130, 128), (33, 1024), (5, 8192)):
        x = (torch.randn((n, row), generator=torch.Generator().manual_seed(n)) * 3).to(torch.bfloat16).to(DEV)
        codes = Guarded((n, row), torch.uint8, fill=0x55)
        scale = Guarded((n,), torch.float32, fill=-1.0)
        _twice(lambda: idxc.quantize_e4m3(x, codes.t, scale.t), [codes, scale], f"quantiser {n}x{row}")
        # scatter into the last rows of a larger cache: only those rows change
        rows = n + 7
        cache = Guarded((rows, row), torch.uint8, fill=0x55)
        cscale = Guarded((rows,), torch.float32, fill=-1.0)
        dst = (torch.arange(n, device=DEV) + 7).to(torch.int64)
        _twice(lambda: idxc.quantize_e4m3(x, cache.t, cscale.t, dst_rows=dst), [cache, cscale], "quantiser append")
        assert torch.equal(cache.t[7:], codes.t) and torch.equal(cscale.t[7:], scale.t)


def test_overlap_and_distillation_loss():
    rows, k_top = 333, 48
    g = torch.Generator().manual_seed(4)
    tops = []
    for _ in range(3):
        t = torch.rand((rows, 6 * k_top), generator=g).topk(k_top, dim=1).indices.to(torch.int32)
        t = torch.sort(t, dim=1).values
        t[::9, k_top // 2:] = -1
        tops.append(t.contiguous().to(DEV))
    a = idxc.topk_overlap(tops)
    b = idxc.topk_overlap(tops)
    assert torch.allclose(a, b, rtol=1e-12, atol=0)                # sums over the rows are fp64 atomics: order may differ
    m, per_row = idxc.topk_overlap(tops[:2], pairs=[(0, 1)], want_rows=True)
    m2, per_row2 = idxc.topk_overlap(tops[:2], pairs=[(0, 1)], want_rows=True)
    assert torch.equal(per_row, per_row2)
    L = 257
    ld = 260
    scores = torch.randn((L, ld), generator=g).to(DEV)
    targets = []
    for _ in range(5):
        p = torch.rand((L, ld), generator=g) * torch.tril(torch.ones(L, ld))
        targets.append((p / p.sum(dim=1, keepdim=True)).to(DEV).contiguous())
    l1, r1 = idxc.distill_kl(scores, targets, want_rows=True)
    l2, r2 = idxc.distill_kl(scores, targets, want_rows=True)
    idxc.poll_device_status()
    assert torch.equal(r1, r2)                      # per-row values are computed by one block each: deterministic
    assert abs(l1.item() - l2.item()) <= 1e-12 * abs(l1.item())     # the total is an fp64 atomic sum over the rows


@pytest.mark.parametrize("n_q,h,k_top", [(3, 128, 200), (70, 16, 65), (149, 128, 130)])
def test_sparse_attention_outputs_and_workspace(n_q, h, k_top):
    n_kv = 1500
    inp = synth.attention_inputs(n_q, n_kv, h, 576, seed=77 + n_q, device=DEV)
    topk = torch.randint(0, n_kv, (n_q, k_top), generator=torch.Generator().manual_seed(n_q), dtype=torch.int32).to(DEV)
    topk[::4, k_top // 3:] = -1
    need = int(idxc.lib().idxc_sparse_attention_workspace_bytes(n_q, k_top))
    ws = Guarded((need,), torch.uint8)
    out = Guarded((n_q, h, 512), torch.bfloat16, fill=7.0)
    got = {}

    def run():
        got["lse"] = idxc.sparse_attention(inp.q, inp.kv, topk, 512, 0.05, out=out.t, workspace=ws.t)[1]
    run()
    lse1 = got["lse"].clone()
    _twice(run, [out], "sparse attention")
    ws.check("sparse attention workspace")
    assert torch.equal(got["lse"], lse1)
