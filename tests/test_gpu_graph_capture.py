"""The indexer calls inside a CUDA graph.

A serving loop captures its decode step once and replays it (the step's two kernels are short enough that launch cost
and the gap between them are a tenth of the step). The library's prefill and decode calls only enqueue kernels on the
caller's stream: no allocation, no synchronisation, no host read of device data. So a captured call must replay to the
same indices as the eager call, and a replay must follow the CONTENTS of its input buffers, not what they held at
capture time.
"""
import pytest
import torch

from paper_2603_12201_b200 import binding as idxc
from paper_2603_12201_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _capture(fn):
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    with torch.cuda.stream(side):
        fn()                                            # warm-up outside the capture (first-use set-up of the library)
        with torch.cuda.graph(g, stream=side):
            fn()
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    return g


@pytest.mark.parametrize("fp8", [False, True])
def test_decode_step_replays_from_a_graph_and_follows_its_buffers(fp8):
    lens = [40000, 17000, 300, 20000, 2048, 131072]     # cluster select, short rows, one row of exactly k_top scores
    B, H, d, k_top = len(lens), 64, 128, 2048
    xa = synth.decode_inputs(B, H, d, 0, 0, seed=71, device=DEV, fp8=fp8, lens=lens)
    xb = synth.decode_inputs(B, H, d, 0, 0, seed=72, device=DEV, fp8=fp8, lens=lens)
    ws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, xa.max_len, H, d, k_top, idxc.FP8_E4M3 if fp8 else idxc.BF16), DEV)

    def eager(x):
        out = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
        idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, x.q_scale, x.k_scale,
                            topk_out=out, workspace=ws)
        torch.cuda.synchronize()
        return out

    want_a, want_b = eager(xa), eager(xb)
    assert not torch.equal(want_a, want_b)
    # the graph reads live buffers that first hold set a, then set b
    q, w = xa.q_step.clone(), xa.w.clone()
    k = xa.k_cache.clone()
    qs = xa.q_scale.clone() if fp8 else None
    ks = xa.k_scale.clone() if fp8 else None
    out = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    g = _capture(lambda: idxc.indexer_decode(q, k, w, xa.k_offsets, xa.lens, xa.max_len, k_top, qs, ks, topk_out=out, workspace=ws))
    out.fill_(-7)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want_a)
    q.copy_(xb.q_step); w.copy_(xb.w); k.copy_(xb.k_cache)
    if fp8:
        qs.copy_(xb.q_scale); ks.copy_(xb.k_scale)
    out.fill_(-7)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want_b)
    idxc.poll_device_status()


def test_prefill_call_replays_from_a_graph():
    L, H, d, k_top = 1500, 64, 128, 256
    inp = synth.prefill_inputs(L, H, d, seed=73, device=DEV)
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H, d, k_top), DEV)
    want = torch.full((L, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, topk_out=want, workspace=ws)
    torch.cuda.synchronize()
    out = torch.full((L, k_top), -7, dtype=torch.int32, device=DEV)
    g = _capture(lambda: idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, topk_out=out, workspace=ws))
    out.fill_(-7)
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(out, want)
    idxc.poll_device_status()
