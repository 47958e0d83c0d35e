"""Seeded synthetic inputs shaped like the paper's indexer workloads.

This module holds NO arithmetic of the method (no scores, no selection): it only
draws random tensors and rounds them to the storage formats. It serves both the
CUDA path and the CPU oracle (through the tests and the benchmark), and imports
neither. The bytes it returns are authoritative: whoever checks a result reads
back exactly these bytes.

Recipes (the paper's own inputs are a 30B model's activations at 10K-200K
context, Sec. 4.2; these stand in for them with the same shapes: k = 2048
selected tokens, long contexts, FP8 indexer, 47/48 layers, 1/4 retention):
  q, k   ~ N(0, 1), stored as bf16, or as e4m3 codes with one fp32 scale per token
  w      ~ N(0, sigma = 1/sqrt(H_I)), fp32
  clustered keys: 16 shared directions c_j ~ N(0, I); id[s] ~ U{0..15};
           k[s] = (c_id[s] + eps_s) / sqrt(2), eps_s ~ N(0, I)
  decode lens ~ U{lo..hi}; each sequence's keys are contiguous rows of one cache buffer
Each tensor draws from its own generator seeded by (seed, layer, tensor id), on
the device asked for; CPU and CUDA streams differ, so a case is defined by
(recipe, seed, device kind).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import torch

E4M3_MAX = 448.0

_TENSOR_IDS = {"q": 1, "k": 2, "w": 3, "centers": 4, "ids": 5, "lens": 6, "attn_q": 7, "attn_kv": 8, "sel": 9}


def _gen(seed: int, layer: int, name: str, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1_000_003 + layer) * 64 + _TENSOR_IDS[name])
    return g


def _randn(shape, gen, device) -> torch.Tensor:
    return torch.randn(shape, generator=gen, device=device, dtype=torch.float32)


def quantize_e4m3(x: torch.Tensor):
    """Per-token e4m3 codes and fp32 scales: scale = max(amax, 1e-12) / 448 over the
    token's trailing dims, value / scale rounded to nearest even, saturating."""
    flat = x.reshape(x.shape[0], -1)
    amax = flat.abs().amax(dim=1).clamp_min(1e-12)
    scale = (amax / E4M3_MAX).to(torch.float32)
    y = (flat / scale[:, None]).clamp_(-E4M3_MAX, E4M3_MAX)
    return y.to(torch.float8_e4m3fn).reshape(x.shape), scale


@dataclass
class PrefillInputs:
    q: torch.Tensor                 # [L, H, d] bf16 or float8_e4m3fn
    k: torch.Tensor                 # [L, d]
    w: torch.Tensor                 # [L, H] fp32
    q_scale: torch.Tensor | None    # [L] fp32 (fp8 only)
    k_scale: torch.Tensor | None    # [L] fp32 (fp8 only)
    fp8: bool


def prefill_inputs(L: int, H: int, d: int, seed: int, device="cpu", layer: int = 0, fp8: bool = False,
                   clustered: bool = False, n_clusters: int = 16) -> PrefillInputs:
    dev = torch.device(device)
    # q is the big one (L*H*d); draw and round it in slabs to bound the fp32 transient
    gq = _gen(seed, layer, "q", dev)
    store = torch.float8_e4m3fn if fp8 else torch.bfloat16
    q = torch.empty((L, H, d), dtype=store, device=dev)
    q_scale = torch.empty((L,), dtype=torch.float32, device=dev) if fp8 else None
    slab = max(1, min(L, (1 << 28) // (H * d)))
    for r0 in range(0, L, slab):
        r1 = min(L, r0 + slab)
        x = _randn((r1 - r0, H, d), gq, dev)
        if fp8:
            q[r0:r1], q_scale[r0:r1] = quantize_e4m3(x)
        else:
            q[r0:r1] = x.to(torch.bfloat16)
        del x
    gk = _gen(seed, layer, "k", dev)
    kf = _randn((L, d), gk, dev)
    if clustered:
        centers = _randn((n_clusters, d), _gen(seed, layer, "centers", dev), dev)
        ids = torch.randint(0, n_clusters, (L,), generator=_gen(seed, layer, "ids", dev), device=dev)
        kf = (centers[ids] + kf) / math.sqrt(2.0)
    if fp8:
        k, k_scale = quantize_e4m3(kf)
    else:
        k, k_scale = kf.to(torch.bfloat16), None
    w = _randn((L, H), _gen(seed, layer, "w", dev), dev) * (1.0 / math.sqrt(H))
    return PrefillInputs(q, k, w.contiguous(), q_scale, k_scale, fp8)


@dataclass
class DecodeInputs:
    q_step: torch.Tensor            # [B, H, d]
    k_cache: torch.Tensor           # [sum(padded lens), d]; sequence b = rows k_offsets[b] .. +lens[b]-1
    w: torch.Tensor                 # [B, H] fp32
    q_scale: torch.Tensor | None    # [B]
    k_scale: torch.Tensor | None    # [rows of k_cache]
    k_offsets: torch.Tensor         # [B] int64 (row units)
    lens: torch.Tensor              # [B] int32
    max_len: int
    fp8: bool


def decode_inputs(B: int, H: int, d: int, len_lo: int, len_hi: int, seed: int, device="cpu", layer: int = 0,
                  fp8: bool = False, lens=None, row_align: int = 128) -> DecodeInputs:
    """One decode step's inputs. Sequence starts are aligned to ``row_align`` cache rows."""
    dev = torch.device(device)
    if lens is None:
        lens_t = torch.randint(len_lo, len_hi + 1, (B,), generator=_gen(seed, layer, "lens", torch.device("cpu")))
    else:
        lens_t = torch.as_tensor(lens, dtype=torch.int64)
        assert lens_t.shape == (B,)
    padded = ((lens_t + row_align - 1) // row_align) * row_align
    offs = torch.zeros(B, dtype=torch.int64)
    if B > 1:
        offs[1:] = torch.cumsum(padded, 0)[:-1]
    rows = int(padded.sum().item())
    xq = _randn((B, H, d), _gen(seed, layer, "q", dev), dev)
    gk = _gen(seed, layer, "k", dev)
    store = torch.float8_e4m3fn if fp8 else torch.bfloat16
    k_cache = torch.empty((rows, d), dtype=store, device=dev)
    k_scale = torch.empty((rows,), dtype=torch.float32, device=dev) if fp8 else None
    slab = 1 << 20
    for r0 in range(0, rows, slab):
        r1 = min(rows, r0 + slab)
        x = _randn((r1 - r0, d), gk, dev)
        if fp8:
            k_cache[r0:r1], k_scale[r0:r1] = quantize_e4m3(x)
        else:
            k_cache[r0:r1] = x.to(torch.bfloat16)
        del x
    if fp8:
        q_step, q_scale = quantize_e4m3(xq)
    else:
        q_step, q_scale = xq.to(torch.bfloat16), None
    w = _randn((B, H), _gen(seed, layer, "w", dev), dev) * (1.0 / math.sqrt(H))
    return DecodeInputs(q_step, k_cache, w.contiguous(), q_scale, k_scale, offs.to(dev), lens_t.to(torch.int32).to(dev),
                        int(lens_t.max().item()) if B else 0, fp8)


@dataclass
class AttnInputs:
    q: torch.Tensor                 # [n_q, H, d_qk] bf16: attention queries
    kv: torch.Tensor                # [n_kv, d_qk] bf16: one shared latent row per token (values = leading columns)


def attention_inputs(n_q: int, n_kv: int, H: int, d_qk: int, seed: int, device="cpu", layer: int = 0) -> AttnInputs:
    """Inputs of the sparse core attention: q, kv ~ N(0, 1) rounded to bf16 (latent rows of a normalised
    cache have unit RMS). No trained weights are involved: the rows are synthetic."""
    dev = torch.device(device)
    gq = _gen(seed, layer, "attn_q", dev)
    q = torch.empty((n_q, H, d_qk), dtype=torch.bfloat16, device=dev)
    slab = max(1, min(n_q, (1 << 28) // (H * d_qk))) if n_q else 1
    for r0 in range(0, n_q, slab):
        r1 = min(n_q, r0 + slab)
        q[r0:r1] = _randn((r1 - r0, H, d_qk), gq, dev).to(torch.bfloat16)
    kv = _randn((n_kv, d_qk), _gen(seed, layer, "attn_kv", dev), dev).to(torch.bfloat16)
    return AttnInputs(q, kv)


def random_selection(positions, k_top: int, seed: int, device="cpu", layer: int = 0) -> torch.Tensor:
    """A stand-in for an indexer's output: for each query position t in ``positions`` a uniformly random set of
    min(k_top, t + 1) distinct causal positions from [0, t], ascending, padded with -1. [len(positions), k_top] int32."""
    dev = torch.device(device)
    pos = torch.as_tensor(positions, dtype=torch.int64, device=dev)
    n = int(pos.max().item()) + 1 if pos.numel() else 0
    g = _gen(seed, layer, "sel", dev)
    out = torch.full((pos.numel(), k_top), -1, dtype=torch.int32, device=dev)
    step = max(1, (1 << 26) // max(n, 1))
    ar = torch.arange(n, device=dev)
    for r0 in range(0, pos.numel(), step):
        p = pos[r0:r0 + step]
        key = torch.rand((p.numel(), n), generator=g, device=dev)
        key.masked_fill_(ar[None, :] > p[:, None], 2.0)                  # not causal: never drawn
        kk = min(k_top, n)
        val, idx = torch.topk(key, kk, dim=1, largest=False)
        idx = torch.where(val <= 1.0, idx, torch.full_like(idx, n + 1))  # fewer than k_top causal positions
        idx, _ = torch.sort(idx, dim=1)
        idx = torch.where(idx > n, torch.full_like(idx, -1), idx)
        # ascending with the -1 padding at the end
        out[r0:r0 + step, :kk] = idx.to(torch.int32)
    return out


def uniform_pattern(n_layers: int, every: int) -> str:
    """Uniform interleaving (Sec. 3.1.1): keep every r-th indexer, e.g. FSSSFSSS... for r = 4."""
    return "".join("F" if l % every == 0 else "S" for l in range(n_layers))


# The five workloads named by the baseline description; sizes only, no data.
CONFIGS = {
    "cfg1": dict(kind="prefill", L=2048, H=16, d=64, k_top=256, seed=0, fp8=False, clustered=False),
    "cfg2": dict(kind="prefill", L=32768, H=64, d=128, k_top=2048, seed=1, fp8=False, clustered=True),
    "cfg3": dict(kind="decode", B=32, H=64, d=128, k_top=2048, len_lo=16384, len_hi=131072, seed=2, fp8=False),
    "cfg4": dict(kind="schedule", N=48, every=4, L=65536, H=64, d=128, k_top=2048, seed=3, fp8=False, clustered=False),
    "cfg5": dict(kind="chunked", N=48, every=4, L=131072, chunk=8192, H=64, d=128, k_top=2048, seed=4, fp8=True,
                 clustered=False, decode_B=8),
}
