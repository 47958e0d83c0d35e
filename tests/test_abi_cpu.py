"""No-GPU checks of the boundary: the shared library loads, exports every symbol the
header declares, validates arguments before touching the device, and its host-side
schedule logic agrees with the schedule oracle and the patterns the paper prints."""
import ctypes
import os
import re

import pytest

from oracle import schedule as oracle_schedule
from tests.test_oracle_schedule import printed_patterns

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def idxc():
    from paper_2603_12201_b200 import build
    build.build()
    from paper_2603_12201_b200 import binding
    return binding


def test_library_exports_every_declared_symbol(idxc):
    header = open(os.path.join(ROOT, "include", "idxc.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = sorted(set(re.findall(r"\b(idxc_[a-z0-9_]+)\s*\(", header)))
    assert declared == sorted(idxc.EXPORTED_SYMBOLS)
    L = idxc.lib()
    for name in declared:
        assert hasattr(L, name), name


def test_status_strings(idxc):
    seen = {idxc.status_string(s) for s in range(7)}
    assert len(seen) == 7 and "ok" in seen


def test_schedule_host_logic_matches_oracle_and_printed_patterns(idxc):
    pats = [p for _, _, _, p in printed_patterns()] + ["F", "FFFF", "FSSSFSSSFSSS"]
    for pat in pats:
        sch = idxc.Schedule(pat)
        want = oracle_schedule.source_layers(pat)
        assert [sch.source(l) for l in range(len(pat))] == want
        assert sch.stats() == (pat.count("F"), pat.count("S"), 0)
        with pytest.raises(idxc.IdxcError):
            sch.source(len(pat))
        sch.close()


@pytest.mark.parametrize("bad", ["", "SFF", "FXS", "fss"])
def test_schedule_rejects_invalid_patterns(idxc, bad):
    with pytest.raises(idxc.IdxcError) as e:
        idxc.Schedule(bad)
    assert e.value.status == idxc.ERR_PATTERN


def test_argument_validation_happens_before_any_device_work(idxc):
    L = idxc.lib()
    one = ctypes.c_void_p(16)      # never dereferenced: the calls must fail on the sizes first
    # k_top out of range
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 16, 64, 0, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 16, 64, 4096, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    # head count / head dim without a tensor-core kernel
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 48, 64, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_UNSUPPORTED
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 16, 96, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_UNSUPPORTED
    # K shorter than the last query position
    assert L.idxc_indexer_prefill(one, one, one, None, None, 4, 8, 8, 16, 64, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    # unknown dtype / flag
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 16, 64, 8, 7, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 16, 64, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0x80, None) == idxc.ERR_INVALID_ARG
    # fp8 without scales, null q, misaligned q
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 64, 128, 8, idxc.FP8_E4M3, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_prefill(None, one, one, None, None, 0, 8, 8, 16, 64, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_prefill(ctypes.c_void_p(20), one, one, None, None, 0, 8, 8, 16, 64, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    # decode: negative batch, missing lens
    assert L.idxc_indexer_decode(one, one, 100, one, None, None, one, one, -1, 10, 16, 64, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_decode(one, one, 100, one, None, None, one, None, 2, 10, 16, 64, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    # top-k: ld not a multiple of 4
    assert L.idxc_topk_rows(one, 10, 2, 1, 1, None, 4, one, None) == idxc.ERR_INVALID_ARG
    # tensor-map row coordinates are 32-bit: (query, head) rows and (sequence, head) rows must stay below 2^31
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 1 << 25, 1 << 25, 64, 128, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_decode(one, one, 100, one, None, None, one, one, 1 << 25, 10, 64, 128, 8, idxc.BF16, None, 0, one, one, 1 << 20, 0, None) == idxc.ERR_INVALID_ARG
    # streaming top-k: index output only, not with the CUDA-core scorer, rows no longer than its position bitmap
    S = idxc.FLAG_STREAM_TOPK
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 64, 128, 8, idxc.BF16, one, 8, one, one, 1 << 20, S, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 64, 128, 8, idxc.BF16, None, 0, None, one, 1 << 20, S, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 8, 64, 128, 8, idxc.BF16, None, 0, one, one, 1 << 20, S | idxc.FLAG_SIMT_SCORER, None) == idxc.ERR_INVALID_ARG
    assert L.idxc_indexer_prefill(one, one, one, None, None, 0, 8, 1 << 19, 64, 128, 8, idxc.BF16, None, 0, one, one, 1 << 20, S, None) == idxc.ERR_UNSUPPORTED



def test_sparse_attention_validation_and_workspace(idxc):
    L = idxc.lib()
    one = ctypes.c_void_p(16)      # never dereferenced
    f = ctypes.c_float(1.0)
    args = lambda **kw: [kw.get("q", one), kw.get("kv", one), kw.get("topk", one), None, kw.get("n_q", 4), kw.get("n_kv", 100),
                         kw.get("H", 128), kw.get("d_qk", 576), kw.get("d_v", 512), kw.get("k_top", 64), f, kw.get("out", one), None,
                         kw.get("ws", one), kw.get("ws_bytes", 1 << 30), None]
    assert L.idxc_sparse_attention(*args(k_top=0)) == idxc.ERR_INVALID_ARG
    assert L.idxc_sparse_attention(*args(n_q=-1)) == idxc.ERR_INVALID_ARG
    assert L.idxc_sparse_attention(*args(d_v=640)) == idxc.ERR_INVALID_ARG          # values wider than the row
    assert L.idxc_sparse_attention(*args(d_qk=512, d_v=512)) == idxc.ERR_UNSUPPORTED
    assert L.idxc_sparse_attention(*args(H=256)) == idxc.ERR_UNSUPPORTED
    assert L.idxc_sparse_attention(*args(q=None)) == idxc.ERR_INVALID_ARG
    assert L.idxc_sparse_attention(*args(out=ctypes.c_void_p(24))) == idxc.ERR_INVALID_ARG   # misaligned
    assert L.idxc_sparse_attention(*args(ws_bytes=64)) == idxc.ERR_WORKSPACE
    assert L.idxc_sparse_attention(*args(n_q=0)) == idxc.OK                          # nothing to do, nothing touched
    # workspace: per-query counts plus the saved probabilities of the resident CTAs (16.5 KB per 64 selected rows)
    assert L.idxc_sparse_attention_workspace_bytes(0, 2048) == 0
    few, many = L.idxc_sparse_attention_workspace_bytes(4, 2048), L.idxc_sparse_attention_workspace_bytes(102400, 2048)
    # 4 queries are split over 8 CTAs each: 32 resident CTAs' scratch plus their fp32 partial results (sized for 128 heads)
    assert few == 256 + 32 * 32 * (16384 + 512) + 4 * 8 * 128 * (512 + 1) * 4    # 4 queries x 8 bytes round up to 256
    assert many == 102400 * 8 + 160 * 32 * (16384 + 512)                            # capped at the largest grid


def test_workspace_queries(idxc):
    assert idxc.prefill_workspace_bytes(0, 0, 16, 64, 8) == 0
    b = idxc.prefill_workspace_bytes(2048, 2048, 16, 64, 256)
    assert b == 2048 * 2048 * 4
    big = idxc.prefill_workspace_bytes(131072, 131072, 64, 128, 2048)
    assert big <= 8 << 30 and big % (131072 * 4 * 32) == 0
    assert idxc.decode_workspace_bytes(32, 131072, 64, 128, 2048) == 32 * 131072 * 4
    # streaming top-k: per row the full scores (rows that are computed again), 9216 candidate slots of 8 bytes, 128 list
    # lengths, sample length, threshold, two flag bytes; plus alignment slack for seven regions
    assert idxc.prefill_workspace_bytes(2048, 2048, 64, 128, 256, idxc.BF16, idxc.FLAG_STREAM_TOPK) == 2048 * (2048 * 4 + 9216 * 8 + 128 + 10) + 7 * 256


def test_binding_refuses_cpu_tensors(idxc):
    import torch
    q = torch.zeros(8, 16, 64, dtype=torch.bfloat16)
    k = torch.zeros(8, 64, dtype=torch.bfloat16)
    w = torch.zeros(8, 16)
    with pytest.raises(ValueError):
        idxc.indexer_prefill(q, k, w, 4, topk_out=torch.zeros(8, 4, dtype=torch.int32))
