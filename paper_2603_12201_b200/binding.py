"""Python binding of the idxc C-ABI library: argument marshalling only.

Every step of the path (scoring, selection, schedule bookkeeping) runs inside
``libidxc.so``; torch is used for device memory and streams. There is no CPU or
eager fallback: if the library is missing or a call fails, an exception is raised.
Function names mirror ``include/idxc.h``.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

import torch

_LIB_PATH = Path(__file__).resolve().parent / "libidxc.so"

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_PATTERN, ERR_CUDA, ERR_DEVICE_TIMEOUT = 1, 2, 3, 4, 5, 6
BF16, FP8_E4M3 = 0, 1
FLAG_COPY_SHARED = 0x1
FLAG_SIMT_SCORER = 0x2
FLAG_FILL_MASKED = 0x4
FLAG_STREAM_TOPK = 0x8

EXPORTED_SYMBOLS = [
    "idxc_status_string", "idxc_prefill_workspace_bytes", "idxc_indexer_prefill", "idxc_decode_workspace_bytes",
    "idxc_indexer_decode", "idxc_topk_rows", "idxc_schedule_create", "idxc_schedule_destroy",
    "idxc_schedule_begin_pass", "idxc_schedule_source", "idxc_schedule_stats", "idxc_schedule_prefill_layer",
    "idxc_schedule_decode_layer", "idxc_poll_device_status", "idxc_launch_count", "idxc_indexer_decode_noalloc",
    "idxc_selftest_bounded_wait", "idxc_selftest_tmem_readout", "idxc_selftest_tmem_readout_under_mma", "idxc_selftest_issue_rates", "idxc_quantize_e4m3", "idxc_topk_overlap", "idxc_pattern_search_dp",
    "idxc_pattern_search_greedy", "idxc_distill_kl", "idxc_sparse_attention_workspace_bytes", "idxc_sparse_attention",
]
NOALLOC_SCRATCH_BYTES = 16 << 20


EVAL_LOSS_FN = ctypes.CFUNCTYPE(ctypes.c_double, ctypes.c_char_p, ctypes.c_int, ctypes.c_void_p)


class IdxcError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it has not been built (run paper_2603_12201_b200/build.py)."""
    global _lib
    if _lib is None:
        if not _LIB_PATH.exists():
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2603_12201_b200.build` "
                               "(there is no fallback path)")
        L = ctypes.CDLL(str(_LIB_PATH))
        vp, i64, i32, u32, sz = ctypes.c_void_p, ctypes.c_int64, ctypes.c_int, ctypes.c_uint32, ctypes.c_size_t
        L.idxc_status_string.restype = ctypes.c_char_p
        L.idxc_status_string.argtypes = [i32]
        L.idxc_launch_count.restype = i64
        L.idxc_prefill_workspace_bytes.restype = sz
        L.idxc_prefill_workspace_bytes.argtypes = [i64, i64, i32, i32, i32, i32, u32]
        L.idxc_decode_workspace_bytes.restype = sz
        L.idxc_decode_workspace_bytes.argtypes = [i32, i64, i32, i32, i32, i32, u32]
        prefill_args = [vp, vp, vp, vp, vp, i64, i64, i64, i32, i32, i32, i32, vp, i64, vp, vp, sz, u32, vp]
        decode_args = [vp, vp, i64, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, vp, i64, vp, vp, sz, u32, vp]
        L.idxc_indexer_prefill.restype = i32
        L.idxc_indexer_prefill.argtypes = prefill_args
        L.idxc_indexer_decode.restype = i32
        L.idxc_indexer_decode.argtypes = decode_args
        L.idxc_indexer_decode_noalloc.restype = i32
        L.idxc_indexer_decode_noalloc.argtypes = [vp, vp, i64, vp, vp, vp, vp, vp, i32, i64, i32, i32, i32, i32, vp, u32, vp]
        L.idxc_topk_rows.restype = i32
        L.idxc_topk_rows.argtypes = [vp, i64, i64, i64, i64, vp, i32, vp, vp]
        L.idxc_schedule_create.restype = i32
        L.idxc_schedule_create.argtypes = [ctypes.c_char_p, i32, ctypes.POINTER(vp)]
        L.idxc_schedule_destroy.restype = None
        L.idxc_schedule_destroy.argtypes = [vp]
        L.idxc_schedule_begin_pass.restype = i32
        L.idxc_schedule_begin_pass.argtypes = [vp]
        L.idxc_schedule_source.restype = i32
        L.idxc_schedule_source.argtypes = [vp, i32, ctypes.POINTER(i32)]
        L.idxc_schedule_stats.restype = i32
        L.idxc_schedule_stats.argtypes = [vp, ctypes.POINTER(i32), ctypes.POINTER(i32), ctypes.POINTER(i64)]
        L.idxc_schedule_prefill_layer.restype = i32
        L.idxc_schedule_prefill_layer.argtypes = [vp, i32] + prefill_args + [ctypes.POINTER(vp)]
        L.idxc_schedule_decode_layer.restype = i32
        L.idxc_schedule_decode_layer.argtypes = [vp, i32] + decode_args + [ctypes.POINTER(vp)]
        L.idxc_topk_overlap.restype = i32
        L.idxc_topk_overlap.argtypes = [vp, vp, i32, i64, i32, vp, vp, vp]
        L.idxc_pattern_search_dp.restype = i32
        L.idxc_pattern_search_dp.argtypes = [vp, i32, i32, ctypes.c_char_p, ctypes.POINTER(ctypes.c_double)]
        L.idxc_pattern_search_greedy.restype = i32
        L.idxc_pattern_search_greedy.argtypes = [i32, i32, EVAL_LOSS_FN, vp, ctypes.c_char_p, ctypes.POINTER(i32),
                                                 ctypes.POINTER(ctypes.c_double), ctypes.POINTER(i64)]
        L.idxc_distill_kl.restype = i32
        L.idxc_distill_kl.argtypes = [vp, i64, i64, i64, i64, ctypes.POINTER(vp), i32, vp, i32, vp, vp, vp]
        L.idxc_sparse_attention_workspace_bytes.restype = sz
        L.idxc_sparse_attention_workspace_bytes.argtypes = [i64, i32]
        L.idxc_sparse_attention.restype = i32
        L.idxc_sparse_attention.argtypes = [vp, vp, vp, vp, i64, i64, i32, i32, i32, i32, ctypes.c_float, vp, vp, vp, sz, vp]
        L.idxc_quantize_e4m3.restype = i32
        L.idxc_quantize_e4m3.argtypes = [vp, i64, i32, vp, vp, vp, vp]
        L.idxc_selftest_bounded_wait.restype = i32
        L.idxc_selftest_bounded_wait.argtypes = [u32, vp]
        L.idxc_selftest_tmem_readout.restype = i32
        L.idxc_selftest_tmem_readout.argtypes = [u32, ctypes.POINTER(i64), vp]
        L.idxc_selftest_tmem_readout_under_mma.restype = i32
        L.idxc_selftest_tmem_readout_under_mma.argtypes = [u32, ctypes.c_int, ctypes.POINTER(i64), vp, vp]
        L.idxc_selftest_issue_rates.restype = i32
        L.idxc_selftest_issue_rates.argtypes = [u32, vp, vp]
        L.idxc_poll_device_status.restype = i32
        L.idxc_poll_device_status.argtypes = [vp]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().idxc_status_string(int(status)).decode()


def launch_count() -> int:
    return int(lib().idxc_launch_count())


def _check(status: int, where: str):
    if status != OK:
        raise IdxcError(status, where)


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _dtype_of(t: torch.Tensor) -> int:
    if t.dtype == torch.bfloat16:
        return BF16
    if t.dtype == torch.float8_e4m3fn:
        return FP8_E4M3
    raise TypeError(f"q/k must be bfloat16 or float8_e4m3fn, got {t.dtype}")


def _dev(t: torch.Tensor, name: str, dtype=None):
    if t is None:
        return None
    if not t.is_cuda:
        raise ValueError(f"{name} must live on a CUDA device (this library has no CPU path)")
    if not t.is_contiguous():
        raise ValueError(f"{name} must be contiguous")
    if dtype is not None and t.dtype != dtype:
        raise TypeError(f"{name}: expected {dtype}, got {t.dtype}")
    return t


def prefill_workspace_bytes(q_len, L_k, H, d, k_top, dt=BF16, flags=0) -> int:
    return int(lib().idxc_prefill_workspace_bytes(q_len, L_k, H, d, k_top, dt, flags))


def decode_workspace_bytes(B, max_len, H, d, k_top, dt=BF16, flags=0) -> int:
    return int(lib().idxc_decode_workspace_bytes(B, max_len, H, d, k_top, dt, flags))


def alloc_workspace(nbytes: int, device) -> torch.Tensor:
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def _prefill_marshal(q, k, w, q_scale, k_scale, q_begin, k_top, scores_out, topk_out, workspace, flags, stream):
    _dev(q, "q"); _dev(k, "k"); _dev(w, "w", torch.float32)
    _dev(q_scale, "q_scale", torch.float32); _dev(k_scale, "k_scale", torch.float32)
    _dev(scores_out, "scores_out", torch.float32); _dev(topk_out, "topk_out", torch.int32); _dev(workspace, "workspace")
    dt = _dtype_of(q)
    if k.dtype != q.dtype:
        raise TypeError("q and k must have the same dtype")
    q_len, H, d = q.shape
    L_k = k.shape[0]
    if k.shape[1] != d or tuple(w.shape) != (q_len, H):
        raise ValueError("shape mismatch between q, k and w")
    ld = 0
    if scores_out is not None:
        if scores_out.dim() != 2 or scores_out.shape[0] != q_len:
            raise ValueError("scores_out must be [q_len, ld]")
        ld = scores_out.shape[1]
    if topk_out is not None and tuple(topk_out.shape) != (q_len, k_top):
        raise ValueError("topk_out must be [q_len, k_top]")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return [_ptr(q), _ptr(k), _ptr(w), _ptr(q_scale), _ptr(k_scale), int(q_begin), q_len, L_k, H, d, int(k_top), dt,
            _ptr(scores_out), ld, _ptr(topk_out), _ptr(workspace), ws_bytes, int(flags), _stream(stream)]


def indexer_prefill(q, k, w, k_top, q_scale=None, k_scale=None, q_begin=0, scores_out=None, topk_out=None,
                    workspace=None, flags=0, stream=None):
    """idxc_indexer_prefill. Writes into scores_out / topk_out (either may be None, not both)."""
    args = _prefill_marshal(q, k, w, q_scale, k_scale, q_begin, k_top, scores_out, topk_out, workspace, flags, stream)
    _check(lib().idxc_indexer_prefill(*args), "idxc_indexer_prefill")


def _decode_marshal(q_step, k_cache, w, q_scale, k_scale, k_offsets, lens, max_len, k_top, scores_out, topk_out,
                    workspace, flags, stream):
    _dev(q_step, "q_step"); _dev(k_cache, "k_cache"); _dev(w, "w", torch.float32)
    _dev(q_scale, "q_scale", torch.float32); _dev(k_scale, "k_scale", torch.float32)
    _dev(k_offsets, "k_offsets", torch.int64); _dev(lens, "lens", torch.int32)
    _dev(scores_out, "scores_out", torch.float32); _dev(topk_out, "topk_out", torch.int32); _dev(workspace, "workspace")
    dt = _dtype_of(q_step)
    if k_cache.dtype != q_step.dtype:
        raise TypeError("q_step and k_cache must have the same dtype")
    B, H, d = q_step.shape
    if k_cache.shape[1] != d or tuple(w.shape) != (B, H) or k_offsets.shape[0] != B or lens.shape[0] != B:
        raise ValueError("shape mismatch between q_step, k_cache, w, k_offsets and lens")
    ld = 0
    if scores_out is not None:
        if scores_out.dim() != 2 or scores_out.shape[0] != B:
            raise ValueError("scores_out must be [B, ld]")
        ld = scores_out.shape[1]
    if topk_out is not None and tuple(topk_out.shape) != (B, k_top):
        raise ValueError("topk_out must be [B, k_top]")
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    return [_ptr(q_step), _ptr(k_cache), k_cache.shape[0], _ptr(w), _ptr(q_scale), _ptr(k_scale), _ptr(k_offsets),
            _ptr(lens), B, int(max_len), H, d, int(k_top), dt, _ptr(scores_out), ld, _ptr(topk_out), _ptr(workspace),
            ws_bytes, int(flags), _stream(stream)]


def indexer_decode(q_step, k_cache, w, k_offsets, lens, max_len, k_top, q_scale=None, k_scale=None, scores_out=None,
                   topk_out=None, workspace=None, flags=0, stream=None):
    """idxc_indexer_decode. ``max_len`` is a host upper bound on ``lens``."""
    args = _decode_marshal(q_step, k_cache, w, q_scale, k_scale, k_offsets, lens, max_len, k_top, scores_out,
                           topk_out, workspace, flags, stream)
    _check(lib().idxc_indexer_decode(*args), "idxc_indexer_decode")


def indexer_decode_noalloc(q_step, k_cache, w, k_offsets, lens, max_len, k_top, topk_out, q_scale=None, k_scale=None,
                           flags=0, stream=None):
    """idxc_indexer_decode_noalloc: the decode step with the score scratch kept in an array
    built into the library, for hosts that cannot hand over (or allocate) a workspace. The
    step's scores, B * round_up(max_len, 32) * 4 bytes, must fit NOALLOC_SCRATCH_BYTES;
    calls that may overlap on the GPU share that array and race."""
    a = _decode_marshal(q_step, k_cache, w, q_scale, k_scale, k_offsets, lens, max_len, k_top, None, topk_out,
                        None, flags, stream)
    # same leading arguments as idxc_indexer_decode, without scores_out/ld and workspace/size
    args = a[:14] + [a[16], a[19], a[20]]
    _check(lib().idxc_indexer_decode_noalloc(*args), "idxc_indexer_decode_noalloc")


def topk_rows(scores, k_top, topk_out, first_len=0, len_step=0, lens=None, stream=None):
    """idxc_topk_rows on a [n_rows, ld] fp32 tensor."""
    _dev(scores, "scores", torch.float32); _dev(topk_out, "topk_out", torch.int32); _dev(lens, "lens", torch.int32)
    n_rows, ld = scores.shape
    if tuple(topk_out.shape) != (n_rows, k_top):
        raise ValueError("topk_out must be [n_rows, k_top]")
    _check(lib().idxc_topk_rows(_ptr(scores), ld, n_rows, int(first_len), int(len_step), _ptr(lens), int(k_top),
                                _ptr(topk_out), _stream(stream)), "idxc_topk_rows")


def quantize_e4m3(x, codes_out, scale_out, dst_rows=None, stream=None):
    """idxc_quantize_e4m3: x [n_tokens, ...] bf16 -> e4m3 codes (float8_e4m3fn or uint8 tensor with the same
    trailing shape) and one fp32 scale per token, written at row r or at row dst_rows[r]."""
    _dev(x, "x", torch.bfloat16); _dev(codes_out, "codes_out"); _dev(scale_out, "scale_out", torch.float32)
    _dev(dst_rows, "dst_rows", torch.int64)
    if codes_out.element_size() != 1:
        raise TypeError("codes_out must be an 8-bit tensor")
    n = x.shape[0]
    row = x.numel() // n if n else int(torch.tensor(x.shape[1:]).prod())
    if codes_out.numel() // max(codes_out.shape[0], 1) != row or scale_out.shape[0] != codes_out.shape[0]:
        raise ValueError("codes_out / scale_out rows do not match x")
    if dst_rows is None and codes_out.shape[0] < n:
        raise ValueError("codes_out has fewer rows than x")
    _check(lib().idxc_quantize_e4m3(_ptr(x), n, row, _ptr(codes_out), _ptr(scale_out), _ptr(dst_rows), _stream(stream)),
           "idxc_quantize_e4m3")


def topk_overlap(layers, pairs=None, want_rows=False, stream=None):
    """idxc_topk_overlap. layers: list of [rows, k_top] int32 index tensors; pairs: list of (a, b) layer
    indices (default: every pair a < b). Returns a [n_pairs] float64 tensor of MEAN row ratios (and, with
    want_rows and a single pair, the per-row ratios)."""
    for t in layers:
        _dev(t, "layer", torch.int32)
    rows, k_top = layers[0].shape
    if pairs is None:
        pairs = [(a, b) for a in range(len(layers)) for b in range(a + 1, len(layers))]
    dev = layers[0].device
    ptrs = torch.tensor([t.data_ptr() for t in layers], dtype=torch.int64, device=dev)
    pr = torch.tensor(pairs, dtype=torch.int32, device=dev).reshape(-1)
    mean = torch.empty((len(pairs),), dtype=torch.float64, device=dev)
    row_out = torch.empty((rows,), dtype=torch.float32, device=dev) if want_rows else None
    _check(lib().idxc_topk_overlap(_ptr(ptrs), _ptr(pr), len(pairs), rows, k_top, _ptr(mean), _ptr(row_out), _stream(stream)),
           "idxc_topk_overlap")
    return (mean, row_out) if want_rows else mean


def pattern_search_dp(S, M: int):
    """idxc_pattern_search_dp on a host [N, N] similarity matrix. Returns (pattern, value)."""
    import numpy as np
    S = np.ascontiguousarray(S, dtype=np.float64)
    N = S.shape[0]
    buf = ctypes.create_string_buffer(N)
    val = ctypes.c_double()
    _check(lib().idxc_pattern_search_dp(S.ctypes.data_as(ctypes.c_void_p), N, int(M), buf, ctypes.byref(val)),
           "idxc_pattern_search_dp")
    return buf.raw[:N].decode(), val.value


def pattern_search_greedy(N: int, K: int, eval_loss, want_losses: bool = False):
    """idxc_pattern_search_greedy (Algorithm 1). eval_loss(pattern: str) -> float.
    Returns (pattern, order of flipped layers, number of evaluations[, loss after each step])."""
    cb = EVAL_LOSS_FN(lambda p, n, user: float(eval_loss(p[:n].decode())))
    buf = ctypes.create_string_buffer(N)
    order = (ctypes.c_int * max(K, 1))()
    losses = (ctypes.c_double * max(K, 1))()
    evals = ctypes.c_int64()
    _check(lib().idxc_pattern_search_greedy(N, K, cb, None, buf, order, losses, ctypes.byref(evals)), "idxc_pattern_search_greedy")
    out = (buf.raw[:N].decode(), list(order)[:K], evals.value)
    return out + (list(losses)[:K],) if want_losses else out


def distill_kl(scores, targets, first_len=1, len_step=1, topk=None, want_rows=False, stream=None):
    """idxc_distill_kl: the multi-layer distillation loss (Eq. 1). scores [rows, ld] fp32; targets: list of
    [rows, ld] fp32 distributions; topk: optional [rows, k] int32. Returns the loss as a 1-element float64 device
    tensor (and the per-row values with want_rows)."""
    _dev(scores, "scores", torch.float32); _dev(topk, "topk", torch.int32)
    rows, ld = scores.shape
    for t in targets:
        _dev(t, "target", torch.float32)
        if tuple(t.shape) != (rows, ld):
            raise ValueError("targets must have the shape of scores")
    ptrs = (ctypes.c_void_p * len(targets))(*[t.data_ptr() for t in targets])
    loss = torch.empty((1,), dtype=torch.float64, device=scores.device)
    row_out = torch.empty((rows,), dtype=torch.float32, device=scores.device) if want_rows else None
    k_top = 0 if topk is None else topk.shape[1]
    _check(lib().idxc_distill_kl(_ptr(scores), ld, rows, int(first_len), int(len_step), ptrs, len(targets), _ptr(topk), k_top,
                                 _ptr(loss), _ptr(row_out), _stream(stream)), "idxc_distill_kl")
    return (loss, row_out) if want_rows else loss


def sparse_attention(q, kv, topk, d_v, scale, kv_base=None, want_lse=True, out=None, workspace=None, stream=None):
    """idxc_sparse_attention: attention of q [n_q, H, d_qk] bf16 over the rows of kv [n_kv, d_qk] bf16 named by
    topk [n_q, k_top] int32 (entries < 0 skipped); values are the leading d_v columns of the same rows.
    Returns (out [n_q, H, d_v] bf16, lse [n_q, H] fp32 or None)."""
    _dev(q, "q", torch.bfloat16); _dev(kv, "kv", torch.bfloat16); _dev(topk, "topk", torch.int32)
    _dev(kv_base, "kv_base", torch.int64)
    n_q, H, d_qk = q.shape
    n_kv = kv.shape[0]
    if kv.shape[1] != d_qk or topk.shape[0] != n_q:
        raise ValueError("kv must be [n_kv, d_qk] and topk [n_q, k_top]")
    if out is None:
        out = torch.empty((n_q, H, d_v), dtype=torch.bfloat16, device=q.device)
    lse = torch.empty((n_q, H), dtype=torch.float32, device=q.device) if want_lse else None
    need = int(lib().idxc_sparse_attention_workspace_bytes(n_q, topk.shape[1]))
    if workspace is None:
        workspace = alloc_workspace(max(need, 256), q.device)
    _check(lib().idxc_sparse_attention(_ptr(q), _ptr(kv), _ptr(topk), _ptr(kv_base), n_q, n_kv, H, d_qk, int(d_v), topk.shape[1],
                                       ctypes.c_float(scale), _ptr(out), _ptr(lse), _ptr(workspace), workspace.numel() * workspace.element_size(),
                                       _stream(stream)), "idxc_sparse_attention")
    return out, lse


def selftest_bounded_wait(wait_cycles: int = 1_000_000, stream=None):
    """idxc_selftest_bounded_wait: enqueue a kernel whose wait can never be satisfied; the next
    poll_device_status() must raise IdxcError(ERR_DEVICE_TIMEOUT)."""
    _check(lib().idxc_selftest_bounded_wait(int(wait_cycles), _stream(stream)), "idxc_selftest_bounded_wait")


def selftest_tmem_readout(accumulators_per_warp: int, stream=None) -> int:
    """idxc_selftest_tmem_readout: enqueue the tensor-memory read-out measurement kernel; returns the accumulator bytes
    the launch reads over all SMs (time the call with CUDA events)."""
    nbytes = ctypes.c_int64()
    _check(lib().idxc_selftest_tmem_readout(int(accumulators_per_warp), ctypes.byref(nbytes), _stream(stream)),
           "idxc_selftest_tmem_readout")
    return int(nbytes.value)


def selftest_tmem_readout_under_mma(accumulators_per_warp: int, fp8: bool, counters, stream=None) -> int:
    """idxc_selftest_tmem_readout_under_mma: the read-out measurement with MMAs running beside it; counters is a device
    int64 tensor of two entries (accumulator fills completed, cycles of the slowest reader). Returns the bytes read."""
    _dev(counters, "counters", torch.int64)
    nbytes = ctypes.c_int64()
    _check(lib().idxc_selftest_tmem_readout_under_mma(int(accumulators_per_warp), int(bool(fp8)), ctypes.byref(nbytes),
                                                      _ptr(counters), _stream(stream)), "idxc_selftest_tmem_readout_under_mma")
    return int(nbytes.value)


ISSUE_RATE_KINDS = ("fmnmx", "fadd_abs", "ffma", "ffma2_packed", "fsetp_sel_pair", "lop3", "shfl")


def selftest_issue_rates(rounds: int = 4096, stream=None) -> dict:
    """idxc_selftest_issue_rates: scheduler cycles per warp instruction for seven instruction kinds (two warps per
    scheduler). Synchronises the stream to read the counters back."""
    s = torch.cuda.current_stream() if stream is None else stream
    cycles = torch.zeros(len(ISSUE_RATE_KINDS), dtype=torch.int64, device=f"cuda:{torch.cuda.current_device()}")
    _check(lib().idxc_selftest_issue_rates(int(rounds), _ptr(cycles), _stream(s)), "idxc_selftest_issue_rates")
    s.synchronize()
    c = cycles.tolist()
    return {name: c[i] / (rounds * (8 if name == "ffma2_packed" else 16) * 2.0) for i, name in enumerate(ISSUE_RATE_KINDS)}


def poll_device_status(stream=None):
    """Synchronises the stream and raises if a kernel recorded a bounded-wait timeout."""
    _check(lib().idxc_poll_device_status(_stream(stream)), "idxc_poll_device_status")


class Schedule:
    """idxc_schedule: the Full/Shared layer pattern and the cached index tensor (host state)."""

    def __init__(self, pattern: str):
        self._h = ctypes.c_void_p()
        self.pattern = pattern
        raw = pattern.encode("ascii", errors="replace")
        _check(lib().idxc_schedule_create(raw, len(raw), ctypes.byref(self._h)), "idxc_schedule_create")
        self._keep = {}          # topk buffers by data_ptr, so a returned alias can be mapped back to its tensor

    def close(self):
        if self._h:
            lib().idxc_schedule_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def begin_pass(self):
        self._keep.clear()
        _check(lib().idxc_schedule_begin_pass(self._h), "idxc_schedule_begin_pass")

    def source(self, layer: int) -> int:
        out = ctypes.c_int()
        _check(lib().idxc_schedule_source(self._h, layer, ctypes.byref(out)), "idxc_schedule_source")
        return out.value

    def stats(self):
        nf, ns, calls = ctypes.c_int(), ctypes.c_int(), ctypes.c_int64()
        _check(lib().idxc_schedule_stats(self._h, ctypes.byref(nf), ctypes.byref(ns), ctypes.byref(calls)),
               "idxc_schedule_stats")
        return nf.value, ns.value, calls.value

    def _result(self, res_ptr, topk_buf):
        if topk_buf is not None:
            self._keep[topk_buf.data_ptr()] = topk_buf
        t = self._keep.get(res_ptr.value)
        if t is None:
            raise RuntimeError("schedule returned a pointer to a buffer this object has not seen")
        return t

    def prefill_layer(self, layer, q=None, k=None, w=None, k_top=0, q_scale=None, k_scale=None, q_begin=0, q_len=None,
                      scores_out=None, topk_buf=None, workspace=None, flags=0, stream=None):
        """One layer of a prefill pass. S layers need only k_top and q_len (inputs may be None).
        Returns the tensor holding this layer's indices (the F layer's buffer on S layers)."""
        res = ctypes.c_void_p()
        if q is None:
            if q_len is None:
                raise ValueError("q_len is required when q is None")
            args = [None, None, None, None, None, int(q_begin), int(q_len), 0, 0, 0, int(k_top), BF16, None, 0,
                    _ptr(_dev(topk_buf, "topk_buf", torch.int32)), None, 0, int(flags), _stream(stream)]
        else:
            args = _prefill_marshal(q, k, w, q_scale, k_scale, q_begin, k_top, scores_out, topk_buf, workspace, flags, stream)
        _check(lib().idxc_schedule_prefill_layer(self._h, layer, *args, ctypes.byref(res)), "idxc_schedule_prefill_layer")
        return self._result(res, topk_buf)

    def decode_layer(self, layer, q_step=None, k_cache=None, w=None, k_offsets=None, lens=None, max_len=0, k_top=0,
                     q_scale=None, k_scale=None, B=None, scores_out=None, topk_buf=None, workspace=None, flags=0,
                     stream=None):
        res = ctypes.c_void_p()
        if q_step is None:
            if B is None:
                raise ValueError("B is required when q_step is None")
            args = [None, None, 0, None, None, None, None, None, int(B), int(max_len), 0, 0, int(k_top), BF16, None, 0,
                    _ptr(_dev(topk_buf, "topk_buf", torch.int32)), None, 0, int(flags), _stream(stream)]
        else:
            args = _decode_marshal(q_step, k_cache, w, q_scale, k_scale, k_offsets, lens, max_len, k_top, scores_out,
                                   topk_buf, workspace, flags, stream)
        _check(lib().idxc_schedule_decode_layer(self._h, layer, *args, ctypes.byref(res)), "idxc_schedule_decode_layer")
        return self._result(res, topk_buf)
