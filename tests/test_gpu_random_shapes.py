"""Seeded random shapes through every device entry point. Prefill and decode: every accepted (H_I, d_I, dtype), ragged lengths,
query chunks against a longer K, workspaces that force chunking, the streaming top-k, empty sequences, unaligned cache
offsets. Each case is checked against the FP64 oracle on sampled rows and against the GPU's own scores (exact top-k with
the lowest-index tie rule); the score-less and streaming paths must give the ordinary path's indices."""
import numpy as np
import pytest
import torch

import oracle
from oracle import distill as odist
from oracle import pattern as opat
from paper_2603_12201_b200 import binding as idxc
from paper_2603_12201_b200 import synth
from tests.util import RTOL_BF16, RTOL_FP8, assert_scores_close, assert_topk_valid, codes, f32

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
SHAPES = [(16, 64, False), (32, 64, False), (64, 64, False), (16, 128, False), (32, 128, False), (64, 128, False),
          (16, 128, True), (32, 128, True), (64, 128, True)]


def to_dev(inp):
    for name in ("q", "k", "w", "q_scale", "k_scale", "q_step", "k_cache", "k_offsets", "lens"):
        if hasattr(inp, name) and getattr(inp, name) is not None:
            setattr(inp, name, getattr(inp, name).to(DEV))
    return inp


def own_exact(g_scores, g_topk, rows, k_top, q_begin):
    for r in rows:
        n = q_begin + r + 1
        kk = min(k_top, n)
        order = np.argsort(-g_scores[r, :n].astype(np.float64), kind="stable")
        assert np.array_equal(np.sort(order[:kk]), g_topk[r, :kk]), f"own top-k row {r}"
        assert np.all(g_topk[r, kk:] == -1), f"tail row {r}"


def prefill_case(rng, i, note):
    H, d, fp8 = SHAPES[rng.integers(len(SHAPES))]
    L = int(rng.choice([rng.integers(1, 300), rng.integers(300, 3000), rng.integers(3000, 9000)]))
    k_top = int(rng.choice([rng.integers(1, 64), rng.integers(64, 1024), 2048, rng.integers(1024, 2049)]))
    q0 = 0 if rng.random() < 0.4 else int(rng.integers(0, L))
    q1 = L if rng.random() < 0.5 else int(rng.integers(q0 + 1, L + 1))
    desc = f"prefill L={L} H={H} d={d} fp8={fp8} k={k_top} q=[{q0},{q1})"
    note["case"] = desc
    inp = to_dev(synth.prefill_inputs(L, H, d, seed=1000 + i, fp8=fp8))
    q, w = inp.q[q0:q1].contiguous(), inp.w[q0:q1].contiguous()
    qs = None if inp.q_scale is None else inp.q_scale[q0:q1].contiguous()
    n = q1 - q0
    ld = (L + 3) // 4 * 4
    scores = torch.full((n, ld), float("nan"), device=DEV)
    topk = torch.full((n, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.indexer_prefill(q, inp.k, w, k_top, qs, inp.k_scale, q_begin=q0, scores_out=scores, topk_out=topk)
    idxc.poll_device_status()
    dt = idxc.FP8_E4M3 if fp8 else idxc.BF16
    # scoreless path, with a workspace that forces chunks sometimes
    full = idxc.prefill_workspace_bytes(n, L, H, d, k_top, dt, 0)
    ws_bytes = full if rng.random() < 0.5 else max(full // int(rng.integers(2, 6)), 1)
    topk2 = torch.full((n, k_top), -7, dtype=torch.int32, device=DEV)
    try:
        idxc.indexer_prefill(q, inp.k, w, k_top, qs, inp.k_scale, q_begin=q0, topk_out=topk2, workspace=idxc.alloc_workspace(ws_bytes, DEV))
        idxc.poll_device_status()
        assert torch.equal(topk, topk2), "scoreless path differs"
    except idxc.IdxcError as e:
        if e.status != idxc.ERR_WORKSPACE:
            raise
    # streaming path
    fl = idxc.FLAG_STREAM_TOPK
    fulls = idxc.prefill_workspace_bytes(n, L, H, d, k_top, dt, fl)
    ws_bytes = fulls if rng.random() < 0.5 else max(fulls // int(rng.integers(2, 6)), 1)
    topk3 = torch.full((n, k_top), -7, dtype=torch.int32, device=DEV)
    try:
        idxc.indexer_prefill(q, inp.k, w, k_top, qs, inp.k_scale, q_begin=q0, topk_out=topk3, workspace=idxc.alloc_workspace(ws_bytes, DEV), flags=fl)
        idxc.poll_device_status()
        assert torch.equal(topk, topk3), "streaming path differs"
    except idxc.IdxcError as e:
        if e.status not in (idxc.ERR_WORKSPACE, idxc.ERR_INVALID_ARG):
            raise
    g_s, g_t = scores.cpu().numpy(), topk.cpu().numpy()
    rows = sorted(set(int(x) for x in rng.integers(0, n, size=min(n, 24))) | {0, n - 1})
    own_exact(g_s, g_t, rows, k_top, q0)
    # nothing right of the diagonal
    for r in rows:
        assert np.all(np.isnan(g_s[r, q0 + r + 1:])), f"row {r} wrote past the diagonal"
    orows = rows[:: max(1, len(rows) // 6)]
    o_scores, _ = oracle.indexer_prefill(codes(q), codes(inp.k), f32(w), k_top, oracle.FP8_E4M3 if fp8 else oracle.BF16,
                                         f32(qs), f32(inp.k_scale), q_begin=q0, rows=orows)
    rtol = RTOL_FP8 if fp8 else RTOL_BF16
    for j, r in enumerate(orows):
        t = q0 + r
        assert_scores_close(g_s[r, : t + 1], o_scores[j, : t + 1], rtol, what=f"row {r}")
        assert_topk_valid(g_t[r], o_scores[j, : t + 1], k_top, rtol, what=f"row {r}")
    return desc


def decode_case(rng, i, note):
    H, d, fp8 = SHAPES[rng.integers(len(SHAPES))]
    B = int(rng.choice([1, 2, rng.integers(1, 9), rng.integers(9, 48)]))
    hi = int(rng.choice([300, 5000, 40000, 140000])) if B <= 8 else int(rng.choice([300, 5000, 20000]))
    lens = [int(x) for x in rng.integers(0, hi + 1, size=B)]
    if rng.random() < 0.3:
        lens[int(rng.integers(B))] = 0
    k_top = int(rng.choice([rng.integers(1, 64), rng.integers(64, 1024), 2048]))
    align = int(rng.choice([1, 8, 128]))
    desc = f"decode B={B} H={H} d={d} fp8={fp8} k={k_top} align={align} lens={lens[:6]}..."
    note["case"] = desc
    inp = to_dev(synth.decode_inputs(B, H, d, 0, 0, seed=5000 + i, fp8=fp8, lens=lens, row_align=align))
    if inp.max_len == 0:
        return desc + " (skipped: all empty)"
    ld = (inp.max_len + 3) // 4 * 4
    scores = torch.full((B, ld), float("nan"), device=DEV)
    topk = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    idxc.indexer_decode(inp.q_step, inp.k_cache, inp.w, inp.k_offsets, inp.lens, inp.max_len, k_top, inp.q_scale,
                        inp.k_scale, scores_out=scores, topk_out=topk)
    idxc.poll_device_status()
    topk2 = torch.full((B, k_top), -7, dtype=torch.int32, device=DEV)
    dt = idxc.FP8_E4M3 if fp8 else idxc.BF16
    ws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, inp.max_len, H, d, k_top, dt), DEV)
    idxc.indexer_decode(inp.q_step, inp.k_cache, inp.w, inp.k_offsets, inp.lens, inp.max_len, k_top, inp.q_scale,
                        inp.k_scale, topk_out=topk2, workspace=ws)
    idxc.poll_device_status()
    assert torch.equal(topk, topk2), "workspace path differs"
    g_s, g_t = scores.cpu().numpy(), topk.cpu().numpy()
    o_scores, _ = oracle.indexer_decode(codes(inp.q_step), codes(inp.k_cache), f32(inp.w), inp.k_offsets.cpu().numpy(),
                                        inp.lens.cpu().numpy(), k_top, oracle.FP8_E4M3 if fp8 else oracle.BF16,
                                        f32(inp.q_scale), f32(inp.k_scale))
    rtol = RTOL_FP8 if fp8 else RTOL_BF16
    for b in range(B):
        n = lens[b]
        assert_scores_close(g_s[b, :n], o_scores[b, :n], rtol, what=f"seq {b}")
        assert np.all(np.isnan(g_s[b, n:])), f"seq {b} wrote past its length"
        assert_topk_valid(g_t[b], o_scores[b, :n], k_top, rtol, what=f"seq {b}")
        order = np.argsort(-g_s[b, :n].astype(np.float64), kind="stable")
        kk = min(k_top, n)
        assert np.array_equal(np.sort(order[:kk]), g_t[b, :kk]), f"own top-k seq {b}"
        assert np.all(g_t[b, kk:] == -1)
    return desc


@pytest.mark.parametrize("seed", [1, 2, 3, 4])
def test_random_shapes(seed):
    rng = np.random.default_rng(seed)
    note = {}
    for i in range(60):
        fn = prefill_case if i % 2 else decode_case
        try:
            fn(rng, 100 * seed + i, note)
        except (AssertionError, idxc.IdxcError) as e:
            raise AssertionError(f"seed {seed} case {i} ({note.get('case')}): {e}") from e


def make_scores(rng, g, n_rows, ld, kind):
    if kind == "normal":
        x = torch.randn((n_rows, ld), device=DEV, generator=g)
    elif kind == "uniform":
        x = torch.rand((n_rows, ld), device=DEV, generator=g)
    elif kind == "relu":       # half of the scores exactly zero
        x = torch.relu(torch.randn((n_rows, ld), device=DEV, generator=g))
    elif kind == "cauchy":
        x = torch.tan(3.14159 * (torch.rand((n_rows, ld), device=DEV, generator=g) - 0.5)).clamp(-1e30, 1e30)
    elif kind == "quant":      # few distinct values
        x = torch.randint(0, int(rng.integers(2, 40)), (n_rows, ld), device=DEV, generator=g).float()
    elif kind == "asc":
        x = torch.arange(ld, device=DEV).float().repeat(n_rows, 1) * 0.25 + torch.randn((n_rows, 1), device=DEV, generator=g)
    elif kind == "desc":
        x = -torch.arange(ld, device=DEV).float().repeat(n_rows, 1) * 0.25
    elif kind == "spike":      # constant with a few outliers
        x = torch.full((n_rows, ld), 1.5, device=DEV)
        m = torch.rand((n_rows, ld), device=DEV, generator=g) < 0.001
        x[m] = torch.randn((int(m.sum()),), device=DEV, generator=g) * 100
    elif kind == "tiny":       # denormals and signed zeros
        x = torch.randn((n_rows, ld), device=DEV, generator=g) * 1e-41
        x[torch.rand((n_rows, ld), device=DEV, generator=g) < 0.2] = -0.0
    elif kind == "huge":
        x = torch.randn((n_rows, ld), device=DEV, generator=g) * 1e37
    elif kind == "bimodal":
        x = torch.randn((n_rows, ld), device=DEV, generator=g) + 50.0 * (torch.rand((n_rows, ld), device=DEV, generator=g) < float(rng.random())).float()
    elif kind == "lognormal":
        x = torch.exp(3 * torch.randn((n_rows, ld), device=DEV, generator=g))
    elif kind == "bf16":       # scores rounded to 8 bits of mantissa: many ties
        x = torch.randn((n_rows, ld), device=DEV, generator=g).bfloat16().float()
    return x.contiguous()


SCORE_KINDS = ["normal", "uniform", "relu", "cauchy", "quant", "asc", "desc", "spike", "tiny", "huge", "bimodal", "lognormal", "bf16"]


def rows_not_exact(x, topk, lens, k_top):
    """Rows whose indices are not the exact top-k (larger score first, lower index first among equal scores, -0 == +0;
    ascending indices, -1 beyond the row's length), by a stable library sort on the GPU."""
    n_rows, ld = x.shape
    col = torch.arange(ld, device=DEV)
    xm = torch.where(col[None, :] < lens[:, None], x, torch.full_like(x, float("-inf")))
    xm = torch.where(xm == 0, torch.zeros_like(xm), xm)          # -0 == +0
    order = torch.sort(xm, dim=1, descending=True, stable=True).indices[:, :k_top]
    if order.shape[1] < k_top:
        order = torch.nn.functional.pad(order, (0, k_top - order.shape[1]), value=0)
    kk = torch.clamp(lens, max=k_top)
    j = torch.arange(k_top, device=DEV)
    valid = j[None, :] < kk[:, None]
    want = torch.where(valid, order, torch.full_like(order, ld + 1))
    want = torch.sort(want, dim=1).values
    want = torch.where(valid, want, torch.full_like(want, -1)).int()
    bad = (want != topk).any(dim=1)
    return bad


def test_topk_rows_adversarial_distributions():
    """The select alone on score distributions chosen against its sampling step: heavy tails, a few distinct values,
    sorted rows, constants with outliers, denormals and signed zeros, values near the float range's end; as a prefill
    chunk (lengths growing by 0, 1 or 2 per row), as a decode step (few rows up to 600K scores) and as many ragged rows."""
    rng = np.random.default_rng(7)
    g = torch.Generator(device=DEV); g.manual_seed(11)
    for i in range(400):
        kind = SCORE_KINDS[rng.integers(len(SCORE_KINDS))]
        mode = int(rng.integers(3))
        k_top = int(rng.choice([1, rng.integers(1, 100), rng.integers(100, 2048), 2048]))
        if mode == 0:
            n_rows = int(rng.integers(1, 3000)); first = int(rng.integers(1, 70000)); step = int(rng.integers(0, 3))
            n_rows = max(1, min(n_rows, int(2e8 // (first + step * n_rows))))
            ld = (first + step * (n_rows - 1) + 3) // 4 * 4
            lens_t = (first + step * torch.arange(n_rows, device=DEV)).int(); args = dict(first_len=first, len_step=step)
        else:
            if mode == 1:
                n_rows = int(rng.integers(1, 140)); hi = int(rng.choice([3000, 40000, 200000, 600000]))
            else:
                n_rows = int(rng.integers(1, 5000)); hi = int(rng.choice([500, 5000, 30000]))
            n_rows = max(1, min(n_rows, int(2e8 // hi)))
            lens_np = rng.integers(0, hi + 1, size=n_rows); ld = max((int(lens_np.max()) + 3) // 4 * 4, 4)
            lens_t = torch.tensor(lens_np, dtype=torch.int32, device=DEV); args = dict(lens=lens_t)
        x = make_scores(rng, g, n_rows, ld, kind)
        topk = torch.full((n_rows, k_top), -7, dtype=torch.int32, device=DEV)
        idxc.topk_rows(x, k_top, topk, **args)
        idxc.poll_device_status()
        bad = rows_not_exact(x, topk, lens_t.long(), k_top)
        assert not bool(bad.any()), f"case {i} {kind} mode {mode} rows {n_rows} ld {ld} k {k_top}: rows {torch.nonzero(bad).flatten()[:5].tolist()}"
        if i % 50 == 0 and int(lens_t.max()) > 0:
            # the checker itself: one spoiled entry must be reported, for its row only
            r = int(torch.argmax(lens_t))
            spoiled = topk.clone()
            spoiled[r, 0] = -1
            bad = rows_not_exact(x, spoiled, lens_t.long(), k_top)
            assert bool(bad[r]) and int(bad.sum()) == 1
        del x, topk


def quant_case(rng, i):
    n = int(rng.choice([1, rng.integers(1, 50), rng.integers(50, 3000)]))
    shape = [(128,), (64,), (256,), (64, 128), (16, 64), (8, 40), (8,), (32, 128), (576,), (24,)][rng.integers(10)]
    desc = f"quant n={n} shape={shape}"
    g = torch.Generator().manual_seed(i)
    mag = torch.exp(torch.randn(n, generator=g) * float(rng.choice([0.1, 3.0, 8.0])))
    x = (torch.randn((n,) + shape, generator=g) * mag[(...,) + (None,) * len(shape)]).to(torch.bfloat16)
    if rng.random() < 0.3:
        x[rng.integers(n)] = 0
    if rng.random() < 0.3:
        x[torch.rand(x.shape, generator=g) < 0.5] = 0
    xd = x.to(DEV)
    codes_out = torch.full((n,) + shape, 0x55, dtype=torch.uint8, device=DEV)
    scale_out = torch.full((n,), -1.0, device=DEV)
    idxc.quantize_e4m3(xd, codes_out, scale_out)
    o_codes, o_scale = oracle.quantize_e4m3(codes(x))
    g_codes = codes_out.cpu().numpy()
    assert np.array_equal(scale_out.cpu().numpy(), o_scale), desc + " scales"
    nz = (o_codes & 0x7F) != 0
    assert np.array_equal(g_codes & 0x7F, o_codes & 0x7F) and np.array_equal(g_codes[nz], o_codes[nz]), desc + " codes"
    return desc


def overlap_case(rng, i):
    n_layers = int(rng.integers(2, 7)); n_rows = int(rng.choice([1, rng.integers(1, 100), rng.integers(100, 3000)]))
    k_top = int(rng.choice([1, rng.integers(1, 64), rng.integers(64, 2049)])); n_keys = int(rng.integers(k_top, 4 * k_top + 50))
    desc = f"overlap layers={n_layers} rows={n_rows} k={k_top} keys={n_keys}"
    tops = []
    for l in range(n_layers):
        key = torch.rand((n_rows, n_keys), device=DEV)
        idx = torch.topk(key, k_top, dim=1).indices.sort(dim=1).values.int()
        # ragged valid counts: -1 tails
        valid = torch.randint(0, k_top + 1, (n_rows,), device=DEV)
        if rng.random() < 0.5:
            idx = torch.where(torch.arange(k_top, device=DEV)[None, :] < valid[:, None], idx, torch.full_like(idx, -1))
        tops.append(idx.contiguous())
    host = [t.cpu().numpy() for t in tops]
    mean = idxc.topk_overlap(tops).cpu().numpy()
    pairs = [(a, b) for a in range(n_layers) for b in range(a + 1, n_layers)]
    for p, (a, b) in enumerate(pairs):
        want = opat.overlap(host[a], host[b])
        assert abs(mean[p] - want) <= 1e-9 or (np.isnan(want) and np.isnan(mean[p])), f"{desc} pair {a},{b}: {mean[p]} vs {want}"
    a, b = int(rng.integers(n_layers)), int(rng.integers(n_layers))
    m1, rows = idxc.topk_overlap(tops, pairs=[(a, b)], want_rows=True)
    want_rows = opat.overlap_rows(host[a], host[b])
    assert np.allclose(rows.cpu().numpy(), want_rows, atol=1e-6, equal_nan=True), desc + " rows"
    return desc


def distill_case(rng, i):
    L = int(rng.choice([1, rng.integers(1, 100), rng.integers(100, 1500)])); n_t = int(rng.integers(1, 8))
    first = int(rng.integers(1, 50)); step = int(rng.integers(0, 2))
    ld = (first + step * (L - 1) + 3) // 4 * 4
    desc = f"distill L={L} targets={n_t} first={first} step={step} ld={ld}"
    gen = torch.Generator().manual_seed(i)
    scores = (torch.randn((L, ld), generator=gen) * float(rng.choice([0.1, 1.0, 10.0]))).to(DEV).contiguous()
    lens = first + step * torch.arange(L)
    mask = (torch.arange(ld)[None, :] < lens[:, None]).float()
    targets = []
    for j in range(n_t):
        p = torch.rand((L, ld), generator=gen) * mask
        if rng.random() < 0.5:
            p = p * (torch.rand((L, ld), generator=gen) < 0.5).float()
            p[:, 0] += 1e-3 * mask[:, 0]
        p = p / p.sum(dim=1, keepdim=True).clamp_min(1e-30)
        targets.append(p.to(DEV).contiguous())
    loss, rows = idxc.distill_kl(scores, targets, first_len=first, len_step=step, want_rows=True)
    want, want_rows = odist.multi_layer_loss(scores.cpu().numpy(), [t.cpu().numpy() for t in targets], first_len=first, len_step=step)
    assert abs(loss.item() - want) <= 2e-5 * abs(want) + 1e-7, f"{desc}: {loss.item()} vs {want}"
    assert np.allclose(rows.cpu().numpy(), want_rows, rtol=1e-4, atol=1e-5), desc + " rows"
    return desc


@pytest.mark.parametrize("seed", [5])
def test_random_shapes_of_the_quantiser_the_overlap_and_the_distillation_loss(seed):
    """Seeded random cases of the three side entry points against their oracles: the quantiser bit for bit (token
    magnitudes over many octaves, zero tokens, half-zero rows, every row width the tests use), the overlap ratios
    (2..6 layers, ragged -1 tails), the distillation loss (1..7 targets, sparse targets, fixed or growing lengths)."""
    rng = np.random.default_rng(seed)
    fns = [quant_case, overlap_case, distill_case]
    for i in range(1, 121):
        fns[i % 3](rng, 1000 * seed + i)
