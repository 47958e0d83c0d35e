"""Two host threads drive the library at the same time, each on a stream of its own.

A server runs prefill chunks and decode steps of different requests from different threads. The library keeps a little
host state (device information, the per-kernel shared-memory opt-in, the launch counter) behind locks and atomics, and
every call works only on its caller's buffers and stream. So whatever the threads interleave, each call must give the
indices it gives alone.
"""
import threading

import pytest
import torch

from paper_2603_12201_b200 import binding as idxc
from paper_2603_12201_b200 import synth

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_prefill_and_decode_from_two_threads_give_their_serial_results():
    H, d, k_top = 64, 128, 512
    # thread A: prefill chunks of one request; thread B: decode steps of another batch (bf16 and e4m3 in turn)
    L = 3000
    pin = synth.prefill_inputs(L, H, d, seed=81, device=DEV)
    pws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(1000, L, H, d, k_top), DEV)
    lens = [20000, 300, 70000, 5000]
    dins = [synth.decode_inputs(len(lens), H, d, 0, 0, seed=82 + i, device=DEV, fp8=bool(i & 1), lens=lens) for i in range(2)]
    dws = [idxc.alloc_workspace(idxc.decode_workspace_bytes(len(lens), x.max_len, H, d, k_top,
                                                            idxc.FP8_E4M3 if i & 1 else idxc.BF16), DEV) for i, x in enumerate(dins)]

    def prefill(out, stream):
        for q0 in range(0, L, 1000):
            sl = slice(q0, min(q0 + 1000, L))
            idxc.indexer_prefill(pin.q[sl], pin.k, pin.w[sl], k_top, q_begin=q0, topk_out=out[sl], workspace=pws, stream=stream)

    def decode(i, out, stream):
        x = dins[i]
        idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, x.q_scale, x.k_scale,
                            topk_out=out, workspace=dws[i], stream=stream)

    cur = torch.cuda.current_stream()
    want_p = torch.full((L, k_top), -7, dtype=torch.int32, device=DEV)
    prefill(want_p, cur)
    want_d = [torch.full((len(lens), k_top), -7, dtype=torch.int32, device=DEV) for _ in range(2)]
    for i in range(2):
        decode(i, want_d[i], cur)
    torch.cuda.synchronize()

    rounds = 12
    got_p = [torch.full((L, k_top), -7, dtype=torch.int32, device=DEV) for _ in range(rounds)]
    got_d = [torch.full((len(lens), k_top), -7, dtype=torch.int32, device=DEV) for _ in range(rounds)]
    sa, sb = torch.cuda.Stream(), torch.cuda.Stream()
    errors = []
    go = threading.Barrier(2)

    def run_a():
        try:
            torch.cuda.set_device(0)
            go.wait()
            for r in range(rounds):
                prefill(got_p[r], sa)
        except Exception as e:                      # noqa: BLE001 (reported by the main thread)
            errors.append(e)

    def run_b():
        try:
            torch.cuda.set_device(0)
            go.wait()
            for r in range(rounds):
                decode(r & 1, got_d[r], sb)
        except Exception as e:                      # noqa: BLE001
            errors.append(e)

    ta, tb = threading.Thread(target=run_a), threading.Thread(target=run_b)
    ta.start(); tb.start()
    ta.join(); tb.join()
    torch.cuda.synchronize()
    assert not errors, errors
    for r in range(rounds):
        assert torch.equal(got_p[r], want_p), f"prefill round {r}"
        assert torch.equal(got_d[r], want_d[r & 1]), f"decode round {r}"
    idxc.poll_device_status()
