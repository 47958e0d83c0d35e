"""Parity of idxc_sparse_attention with the oracle (Sec. 2.1: attention over the selected subset; Fig. 2 SparseAttn).

Tolerance. Scores are exact bf16 products summed in fp32 (error ~1e-6 of the operand norms, negligible). The
probabilities are rounded to bf16 before the second product: independent relative errors, uniform within 2^-9,
standard deviation 2^-9 / sqrt(3) = 1.1e-3, so the output moves by about 1.1e-3 * sqrt(sum_j p_j^2 v_j^2), which is
also the scale of the output row itself (its rms). The output is then rounded to bf16: up to 2^-9 = 2e-3 relative.
Together about 1.6e-3 * rms per output as a standard deviation; the cases below compare several million outputs,
whose largest deviation sits near 5.5 sigma = 9e-3 * rms. The bound used is
|gpu - oracle| <= 1.5e-2 * max(|oracle|, rms of that (query, head) output row), about 9 sigma; an indexing or
masking mistake moves outputs by the order of rms itself. lse is compared to 2e-3 absolute.
"""
import numpy as np
import pytest
import torch

from oracle import sparse_attn as osa
from paper_2603_12201_b200 import binding, synth
from tests.util import codes

pytestmark = pytest.mark.gpu

RTOL_ATTN = 1.5e-2
ATOL_LSE = 2e-3
H, D_QK, D_V = 128, 576, 512


def _check(out, lse, o_out, o_lse, rows, what):
    g = out.float().cpu().numpy()[rows].astype(np.float64)
    rms = np.sqrt(np.mean(np.square(o_out), axis=-1, keepdims=True))
    bound = RTOL_ATTN * np.maximum(np.abs(o_out), rms)
    err = np.abs(g - o_out)
    bad = err > bound
    assert not bad.any(), f"{what}: {int(bad.sum())} outputs off, worst {float((err / np.maximum(bound, 1e-300)).max()):.2f}x the bound at {np.argwhere(bad)[0]}"
    if lse is not None:
        gl = lse.cpu().numpy()[rows].astype(np.float64)
        fin = np.isfinite(o_lse)
        assert np.array_equal(np.isneginf(gl), np.isneginf(o_lse)), f"{what}: lse -inf pattern"
        assert np.all(np.abs(gl[fin] - o_lse[fin]) <= ATOL_LSE), f"{what}: lse off by {np.abs(gl[fin] - o_lse[fin]).max()}"
    return float((err / np.maximum(bound, 1e-300)).max())


def _run(inp, topk, scale, kv_base=None, rows=None, h=H, what=""):
    out, lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, scale, kv_base=kv_base)
    binding.poll_device_status()
    rows = np.arange(inp.q.shape[0]) if rows is None else np.asarray(rows)
    o_out, o_lse = osa.sparse_attention(codes(inp.q), codes(inp.kv), topk.cpu().numpy(), D_V, scale,
                                        kv_base=None if kv_base is None else kv_base.cpu().numpy(), rows=rows)
    return _check(out, lse, o_out, o_lse, rows, what)


def test_prefill_ragged_rows_flat_and_peaked_softmax():
    # positions chosen so that rows hold 1, 63, 64, 65, 127..129, 2047, 2048 entries: several tiles and ragged tails
    pos = [0, 62, 63, 64, 126, 127, 128, 1000, 2046, 2047, 2048, 2500, 2999]
    n_kv = 3000
    inp = synth.attention_inputs(len(pos), n_kv, H, D_QK, seed=11, device="cuda")
    topk = synth.random_selection(pos, 2048, seed=11, device="cuda")
    assert int((topk[3] >= 0).sum()) == 65 and int((topk[-1] >= 0).sum()) == 2048
    _run(inp, topk, 1.0 / np.sqrt(D_QK), what="flat")
    # a large scale makes the softmax peaked: the running reference maximum has to move and O be rescaled
    _run(inp, topk, 0.3, what="peaked")


def test_many_queries_span_all_ctas():
    n_q, n_kv = 400, 4096                      # more queries than SMs: every CTA walks several queries
    pos = torch.randint(0, n_kv, (n_q,), generator=torch.Generator().manual_seed(5)).tolist()
    inp = synth.attention_inputs(n_q, n_kv, H, D_QK, seed=12, device="cuda")
    topk = synth.random_selection(pos, 512, seed=12, device="cuda")
    rows = list(range(0, n_q, 9)) + [n_q - 1]
    _run(inp, topk, 0.08, rows=rows, what="many")


def test_skipped_entries_anywhere_out_of_range_and_empty_rows():
    n_q, n_kv, k_top = 6, 500, 300
    inp = synth.attention_inputs(n_q, n_kv, H, D_QK, seed=13, device="cuda")
    topk = synth.random_selection([499] * n_q, k_top, seed=13, device="cuda")
    g = torch.Generator().manual_seed(1)
    holes = torch.rand((k_top,), generator=g) < 0.3
    topk[0, holes.cuda()] = -1                               # holes anywhere
    topk[1, 64:128] = -1                                     # one whole tile of holes
    topk[2, :] = -1                                          # nothing selected
    topk[3, 10:20] = 100000                                  # outside the cache: skipped
    topk[4] = topk[4].flip(0)                                # order is free
    topk[5, 1:] = -1                                         # a single entry: out = its value row
    out, lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, 0.1)
    binding.poll_device_status()
    o_out, o_lse = osa.sparse_attention(codes(inp.q), codes(inp.kv), topk.cpu().numpy(), D_V, 0.1)
    _check(out, lse, o_out, o_lse, np.arange(n_q), "holes")
    assert torch.all(out[2] == 0) and torch.all(torch.isneginf(lse[2]))
    only = int(topk[5, 0])
    assert torch.equal(out[5], inp.kv[only, :D_V].expand(H, D_V))


def test_rows_outside_the_selection_are_never_read():
    # every cache row that no query selects is filled with NaN: the result must not change (skipped entries stand in
    # with a selected row, never with an arbitrary one)
    n_q, n_kv, k_top = 70, 2000, 200
    inp = synth.attention_inputs(n_q, n_kv, H, D_QK, seed=16, device="cuda")
    g = torch.Generator().manual_seed(3)
    topk = torch.randint(1, n_kv, (n_q, k_top), generator=g, dtype=torch.int32).cuda()      # row 0 is never selected
    topk[:, ::7] = -1
    topk[5, :] = -1
    used = torch.zeros(n_kv, dtype=torch.bool, device="cuda")
    used[topk[topk >= 0].long()] = True
    ref, ref_lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, 0.07)
    poisoned = inp.kv.clone()
    poisoned[~used] = float("nan")
    out, lse = binding.sparse_attention(inp.q, poisoned, topk, D_V, 0.07)
    binding.poll_device_status()
    assert not bool(used[0]) and bool(torch.isnan(poisoned[0]).all())
    assert torch.equal(out, ref) and torch.equal(lse, ref_lse)
    assert bool(torch.isfinite(out.float()).all())


def test_fewer_heads_and_decode_style_base_offsets():
    h, B = 16, 5
    lens = [700, 64, 2100, 1, 300]
    offs = np.concatenate([[0], np.cumsum([((n + 127) // 128) * 128 for n in lens])[:-1]])
    n_kv = int(offs[-1] + lens[-1])
    inp = synth.attention_inputs(B, n_kv, h, D_QK, seed=14, device="cuda")
    topk = synth.random_selection([n - 1 for n in lens], 2048, seed=14, device="cuda")       # relative to the sequence
    base = torch.as_tensor(offs, dtype=torch.int64, device="cuda")
    _run(inp, topk, 0.06, kv_base=base, h=h, what="decode")


def test_indices_from_the_indexer_chain():
    # the real chain: indexer scores -> top-k -> attention over those rows
    L, k_top = 1536, 256
    pin = synth.prefill_inputs(L, 64, 128, seed=15, device="cuda", clustered=True)
    topk = torch.empty((L, k_top), dtype=torch.int32, device="cuda")
    ws = binding.alloc_workspace(binding.prefill_workspace_bytes(L, L, 64, 128, k_top), "cuda")
    binding.indexer_prefill(pin.q, pin.k, pin.w, k_top, topk_out=topk, workspace=ws)
    inp = synth.attention_inputs(L, L, H, D_QK, seed=15, device="cuda")
    rows = [0, 1, 63, 255, 256, 257, 777, L - 1]
    _run(inp, topk, 1.0 / np.sqrt(D_QK), rows=rows, what="chain")


def test_argument_errors():
    inp = synth.attention_inputs(2, 10, H, D_QK, seed=1, device="cuda")
    topk = torch.zeros((2, 8), dtype=torch.int32, device="cuda")
    with pytest.raises(binding.IdxcError) as e:
        binding.sparse_attention(inp.q[:, :, :512].contiguous(), inp.kv[:, :512].contiguous(), topk, 256, 1.0)
    assert e.value.status == binding.ERR_UNSUPPORTED
    with pytest.raises(binding.IdxcError) as e:
        binding.sparse_attention(inp.q, inp.kv, topk, D_V, 1.0, workspace=torch.empty(4, dtype=torch.uint8, device="cuda"))
    assert e.value.status == binding.ERR_WORKSPACE
    # zero queries: nothing to do
    out, _ = binding.sparse_attention(inp.q[:0], inp.kv, topk[:0], D_V, 1.0)
    assert out.shape == (0, H, D_V)


def test_bench_size_chain_sampled_queries():
    # the launch configuration of bench.py's sparse-attention section: the last 8192 queries of an L = 32768 prefill,
    # k_top = 2048, indices from the indexer; the oracle checks a sample of whole queries, the rest is checked for
    # finiteness and against the convex-hull property (|out| cannot exceed the largest selected |value|)
    L, n_q, k_top = 32768, 8192, 2048
    q0 = L - n_q
    pin = synth.prefill_inputs(L, 64, 128, seed=7, device="cuda", clustered=True)
    topk = torch.empty((n_q, k_top), dtype=torch.int32, device="cuda")
    ws = binding.alloc_workspace(binding.prefill_workspace_bytes(n_q, L, 64, 128, k_top), "cuda")
    binding.indexer_prefill(pin.q[q0:], pin.k, pin.w[q0:], k_top, q_begin=q0, topk_out=topk, workspace=ws)
    del pin, ws
    inp = synth.attention_inputs(n_q, L, H, D_QK, seed=7, device="cuda")
    scale = 1.0 / np.sqrt(D_QK)
    out, lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, scale)
    binding.poll_device_status()
    assert bool(torch.isfinite(out.float()).all()) and bool(torch.isfinite(lse).all())
    vmax = float(inp.kv[:, :D_V].float().abs().max())
    assert float(out.float().abs().max()) <= vmax * (1 + 2 ** -7)
    rows = [0, 1, 147, 148, 2047, 4096, n_q - 149, n_q - 1]
    o_out, o_lse = osa.sparse_attention(codes(inp.q[rows]), codes(inp.kv), topk[rows].cpu().numpy(), D_V, scale)
    _check(out, lse, o_out, o_lse, np.asarray(rows), "bench size")


@pytest.mark.parametrize("n_q,n_kv,h,k_top", [(1, 1, 1, 1), (3, 70, 7, 65), (2, 5000, 128, 4096), (149, 64, 33, 64)])
def test_degenerate_shapes(n_q, n_kv, h, k_top):
    # one head, one cache row, k_top below / just above / far above a tile, more selected slots than cache rows
    # (entries repeat: duplicates count twice), one query more than there are SMs
    inp = synth.attention_inputs(n_q, n_kv, h, D_QK, seed=21, device="cuda")
    g = torch.Generator().manual_seed(n_q * 1000 + k_top)
    topk = torch.randint(0, n_kv, (n_q, k_top), generator=g, dtype=torch.int32).cuda()
    _run(inp, topk, 0.05, h=h, what=f"degenerate {n_q}x{n_kv}x{h}x{k_top}")


def test_more_tiles_than_rescale_flags():
    # k_top beyond 256 tiles of 64 entries: the per-tile "rescaled" flags of the second pass cover 256 tiles, later
    # tiles always take the hand-over with the softmax warps; 64 queries so that no query is split over several CTAs
    n_q, n_kv, h, k_top = 64, 900, 4, 16384 + 192
    inp = synth.attention_inputs(n_q, n_kv, h, D_QK, seed=23, device="cuda")
    g = torch.Generator().manual_seed(23)
    topk = torch.randint(0, n_kv, (n_q, k_top), generator=g, dtype=torch.int32).cuda()
    topk[1, 16400:] = -1                                    # ends inside the tiles beyond the flags
    _run(inp, topk, 0.3, rows=[0, 1, 63], h=h, what="259 tiles")


def test_repeated_calls_give_identical_bits():
    # the result does not depend on timing between the roles of the kernel (gather, MMA, softmax, loaders): twenty calls
    # on the same inputs, prefill-style and split (decode-style), agree bit for bit
    for n_q, k_top in ((300, 1024), (24, 2048)):
        n_kv = 6000
        inp = synth.attention_inputs(n_q, n_kv, H, D_QK, seed=31, device="cuda")
        g = torch.Generator().manual_seed(31 + n_q)
        topk = torch.randint(0, n_kv, (n_q, k_top), generator=g, dtype=torch.int32).cuda()
        topk[::5, k_top // 2:] = -1
        ref, ref_lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, 0.2)
        for _ in range(20):
            out, lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, 0.2)
            assert torch.equal(out, ref) and torch.equal(lse, ref_lse)
        binding.poll_device_status()


def test_few_tiles_per_cta_after_unrelated_calls():
    # Split mode with one to four tiles per CTA: the second pass can finish before a softmax warp has looked at the first
    # pass's completion (regression: both completions once shared a barrier and the late warp waited for ever). Calls
    # with full-head queries in between leave different leftovers in shared memory for the 112 head rows this call does
    # not load, which varies the timing of its warps.
    h, B = 16, 5
    lens = [700, 64, 2100, 1, 300]
    offs = np.concatenate([[0], np.cumsum([((n + 127) // 128) * 128 for n in lens])[:-1]])
    n_kv = int(offs[-1] + lens[-1])
    inp = synth.attention_inputs(B, n_kv, h, D_QK, seed=14, device="cuda")
    topk = synth.random_selection([n - 1 for n in lens], 2048, seed=14, device="cuda")
    base = torch.as_tensor(offs, dtype=torch.int64, device="cuda")
    other = synth.attention_inputs(148, 4096, H, D_QK, seed=15, device="cuda")
    other_topk = torch.randint(0, 4096, (148, 256), generator=torch.Generator().manual_seed(15), dtype=torch.int32).cuda()
    ref, ref_lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, 0.06, kv_base=base)
    for _ in range(150):
        binding.sparse_attention(other.q, other.kv, other_topk, D_V, 0.05)
        out, lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, 0.06, kv_base=base)
        assert torch.equal(out, ref) and torch.equal(lse, ref_lse)
    binding.poll_device_status()


@pytest.mark.parametrize("seed", [3, 4])
def test_random_shapes(seed):
    """Seeded random shapes: 1..700 queries (whole and split over CTAs), 1..128 heads, 1..5000 selected slots, caches of
    1..20000 rows, per-query base offsets, holes anywhere, ragged tails, out-of-range entries, flat to peaked softmax;
    sampled queries against the oracle, and a second call must reproduce the first bit for bit."""
    rng = np.random.default_rng(seed)
    for i in range(1, 101):
        n_q = int(rng.choice([rng.integers(1, 8), rng.integers(8, 64), rng.integers(64, 160), rng.integers(160, 700)]))
        n_kv = int(rng.choice([rng.integers(1, 100), rng.integers(100, 3000), rng.integers(3000, 20000)]))
        h = int(rng.choice([1, 16, 64, 128, rng.integers(1, 129)]))
        k_top = int(rng.choice([rng.integers(1, 64), 64, rng.integers(64, 600), 2048, rng.integers(600, 5000)]))
        scale = float(rng.choice([1.0 / 24, 0.02, 0.1, 0.3]))
        desc = f"n_q={n_q} n_kv={n_kv} h={h} k={k_top} scale={scale:.3f}"
        inp = synth.attention_inputs(n_q, n_kv, h, D_QK, seed=100 * seed + i, device="cuda")
        g = torch.Generator().manual_seed(1000 * seed + i)
        use_base = rng.random() < 0.3
        if use_base:
            base_np = rng.integers(0, max(1, n_kv // 2), size=n_q)
            span = n_kv - int(base_np.max())
            topk = torch.randint(0, max(span, 1), (n_q, k_top), generator=g, dtype=torch.int32)
            base = torch.as_tensor(base_np, dtype=torch.int64, device="cuda")
        else:
            topk = torch.randint(0, n_kv, (n_q, k_top), generator=g, dtype=torch.int32)
            base = None
        mode = rng.integers(4)
        if mode == 1:
            topk[torch.rand((n_q, k_top), generator=g) < float(rng.random())] = -1
        elif mode == 2:      # ragged tails like an indexer's output
            for r in range(n_q):
                topk[r, int(rng.integers(0, k_top + 1)):] = -1
        elif mode == 3:      # some out of range entries (skipped)
            topk[torch.rand((n_q, k_top), generator=g) < 0.1] = n_kv + 5
        topk = topk.cuda()
        out, lse = binding.sparse_attention(inp.q, inp.kv, topk, D_V, scale, kv_base=base)
        binding.poll_device_status()
        n_rows = min(n_q, max(1, int(3e8 // (h * k_top * D_QK))))
        rows = np.unique(np.concatenate([[0, n_q - 1], rng.integers(0, n_q, size=n_rows)]))
        o_out, o_lse = osa.sparse_attention(codes(inp.q), codes(inp.kv), topk.cpu().numpy(), D_V, scale,
                                            kv_base=None if base is None else base.cpu().numpy(), rows=rows)
        _check(out, lse, o_out, o_lse, rows, f"seed {seed} case {i}: {desc} mode={mode} base={use_base}")
        out2, lse2 = binding.sparse_attention(inp.q, inp.kv, topk, D_V, scale, kv_base=base)
        assert torch.equal(out, out2) and torch.equal(lse, lse2), f"seed {seed} case {i}: {desc}: second call differs"
