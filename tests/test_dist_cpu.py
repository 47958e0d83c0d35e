"""World-size-2 checks of the multi-GPU measurement plumbing on CPU (gloo): the ranks work on
independent problems, meet at barriers, and the reported time is the slowest rank's."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2603_12201_b200 import dist as pdist
    from paper_2603_12201_b200 import synth
    r, w = pdist.init("gloo")
    assert (r, w) == (rank, world)
    # independent problem per rank: different seeds give different data
    inp = synth.prefill_inputs(16, 16, 64, seed=pdist.rank_seed(7, r))
    digest = float(inp.w.double().sum())
    pdist.barrier(w)
    slowest = pdist.max_over_ranks(10.0 * (r + 1), w)          # rank r "took" 10(r+1) ms
    rate = pdist.whole_job_rate(units_per_rank=100.0, steps=4, slowest_ms=slowest, world=w)
    pdist.barrier(w)
    pdist.shutdown(w)
    out.put((r, slowest, rate, digest))


def test_two_ranks_report_the_slowest_time_and_the_whole_job_rate():
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, out)) for r in range(world)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in results] == [0, 1]
    assert all(r[1] == 20.0 for r in results)                  # max over ranks, on every rank
    assert all(r[2] == pytest.approx(2 * 100.0 * 4 / 20e-3) for r in results)
    assert results[0][3] != results[1][3]                      # the ranks drew different inputs


def test_single_rank_needs_no_process_group():
    from paper_2603_12201_b200 import dist as pdist
    assert pdist.max_over_ranks(3.5, 1) == 3.5
    pdist.barrier(1)
    assert pdist.whole_job_rate(10.0, 2, 4.0, 1) == pytest.approx(5000.0)


def test_attention_input_generators_on_cpu():
    # the seeded generators of the attention step: shapes, dtype, determinism; selections are causal, distinct,
    # ascending and padded with -1
    import torch
    from paper_2603_12201_b200 import synth
    a = synth.attention_inputs(3, 50, 4, 64, seed=5)
    b = synth.attention_inputs(3, 50, 4, 64, seed=5)
    assert a.q.shape == (3, 4, 64) and a.kv.shape == (50, 64) and a.q.dtype == torch.bfloat16
    assert torch.equal(a.q, b.q) and torch.equal(a.kv, b.kv)
    pos = [0, 3, 10, 49]
    sel = synth.random_selection(pos, 8, seed=5)
    assert sel.shape == (4, 8) and sel.dtype == torch.int32
    for t, row in zip(pos, sel.tolist()):
        valid = [x for x in row if x >= 0]
        assert len(valid) == min(8, t + 1) and row[len(valid):] == [-1] * (8 - len(valid))
        assert valid == sorted(set(valid)) and all(0 <= x <= t for x in valid)
    assert torch.equal(sel, synth.random_selection(pos, 8, seed=5))
