#!/usr/bin/env python
"""Benchmark of the lightning-indexer hot path on B200.

One "step" = one Full layer of the indexer on the config-2 workload (L = 32768, H_I = 64,
d_I = 128, k = 2048, clustered keys): the scoring kernel followed by the top-k kernel,
called through the C-ABI binding. The headline `value` is causal (query, key) pairs scored
and selected per second, inputs resident in HBM. The same JSON line also carries
  roofline      the dominant kernel (tcgen05 scorer) against the measured BF16 peak, the top-k kernel
                against the measured HBM bandwidth, and a compact result per workload (`by_config`)
  e2e           the same step with host buffers (pinned H2D of q/k/w, D2H of the indices)
  cpu_baseline  the FP64 oracle timed on the machine's host cores on a bounded row sample
  cfg1          config 1 (L = 2048, H_I = 16, d_I = 64, k = 256): microseconds per call, scores + indices
  decode        config 3 (B = 32, 16K-128K cached keys): microseconds per decode step vs HBM
  schedule      config 4 (N = 48 layers, L = 65536): IndexCache 1-in-4 Full pattern vs all-Full, with checks
  fp8_chunked   config 5 (L = 131072 in 16 chunks, e4m3): one Full layer, the 48-layer schedule, the decode
                step at batch 8 on rotated caches, and both rooflines of the FP8 scorer
plus the steps around the indexer (sparse attention, quantiser, pattern tooling, distillation loss).
Every section carries the SM clock and throttle reasons sampled while it ran. `--quick` shrinks the
extra sections for profiling runs. `--impl reference` times the CPU oracle instead (rank 0 only).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import statistics
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

METRIC = "indexer+top-k Gpairs/s (prefill)"
UNIT = "Gpairs/s"

# Nominal chip figures (dense, no sparsity), for the second fraction of every roofline block.
NOMINAL = {"bf16_tflops": 2250.0, "fp8_tflops": 4500.0, "hbm_gbs": 7700.0, "sm_max_mhz": 1965.0}


def dram_traffic(kernel: str, case: str):
    """dram__bytes_read.sum + dram__bytes_write.sum of one launch of `kernel` on `case`, from the ncu captures
    recorded in profiles/dram_traffic.json (which names the commit each figure was captured at); None if the
    file holds no figure for that kernel and case."""
    try:
        with open(os.path.join(ROOT, "profiles", "dram_traffic.json")) as fh:
            d = json.load(fh)
        e = d["kernels"][kernel][case]
        return int(e["dram_bytes_read"]) + int(e["dram_bytes_write"])
    except Exception:
        return None


def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as fh:
            d = json.load(fh)
        return dict(hbm_gbs=d["hbm_gbs"], bf16_tflops=d["bf16_tflops"],
                    bf16_tflops_sustained=d.get("bf16_tflops_sustained", d["bf16_tflops"]), source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0, source="fallback")


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    def __init__(self, device_index: int, period_s: float = 0.005):
        self.period = period_s
        self.samples = []
        self.reasons = set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            try:
                uuid = torch.cuda.get_device_properties(device_index).uuid
                self._h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + str(uuid)).encode())
            except Exception:
                self._h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self._h = None

    _NAMES = {
        0x2: "applications_clocks_setting", 0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x10: "sync_boost",
        0x20: "sw_thermal_slowdown", 0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown",
        0x100: "display_clock_setting",
    }

    def _run(self):
        nv = self.nv
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h)
                for bit, name in self._NAMES.items():
                    if r & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._run, daemon=True)
            self._thread.start()
        return self

    def reset(self):
        """Forgets what was sampled so far (the sampler keeps running): call at the start of the timed region."""
        self.samples.clear()
        self.reasons.clear()

    def __exit__(self, *exc):
        self._stop.set()
        if self._thread is not None:
            self._thread.join()

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": ["unavailable"]}
        return {"sm_mhz": statistics.median(self.samples), "sm_max_mhz": self.max_mhz, "samples": len(self.samples),
                "reasons": sorted(self.reasons)}


def workload_name(name: str, c: dict) -> str:
    return (f"{name}: single-layer indexer prefill, batch 1, L={c['L']}, H_I={c['H']}, d_I={c['d']}, k_top={c['k_top']}, "
            f"causal, seed {c['seed']}" + (", clustered keys" if c["clustered"] else ""))


def causal_pairs(L: int) -> int:
    return L * (L + 1) // 2


def sample_rows(L: int, n: int, offset: int = 0):
    """Deterministic bounded sample of whole rows: evenly spaced, plus the edges."""
    stride = max(1, L // n)
    rows = sorted(set([0, L - 1] + [min(L - 1, offset % stride + i * stride) for i in range(n)]))
    return rows


def oracle_sample_rate(inp, k_top, rows):
    """Times the oracle (as it stands) on the listed rows; returns (pairs/s, seconds, index rows)."""
    import oracle
    from tests.util import codes, f32
    dt = oracle.FP8_E4M3 if inp.fp8 else oracle.BF16
    q, k, w = codes(inp.q), codes(inp.k), f32(inp.w)
    qs, ks = f32(inp.q_scale), f32(inp.k_scale)
    t0 = time.perf_counter()
    _, tk = oracle.indexer_prefill(q, k, w, k_top, dt, qs, ks, rows=rows, want_scores=False)
    sec = time.perf_counter() - t0
    pairs = sum(r + 1 for r in rows)
    return pairs / sec, sec, tk


def run_reference(args, rank):
    """--impl reference: the CPU oracle on bounded row samples of the same workload."""
    if rank != 0:
        return
    import oracle
    from paper_2603_12201_b200 import synth
    c = synth.CONFIGS[args.workload]
    L, H, d, k_top = c["L"], c["H"], c["d"], c["k_top"]
    inp = synth.prefill_inputs(L, H, d, seed=c["seed"], device="cpu", fp8=c["fp8"], clustered=c["clustered"])
    n_rows = args.ref_rows
    for i in range(args.warmup):
        oracle_sample_rate(inp, k_top, sample_rows(L, max(8, n_rows // 8), offset=i))
    total_pairs, total_sec = 0, 0.0
    for i in range(args.steps):
        rows = sample_rows(L, n_rows, offset=7 * i + 3)
        rate, sec, _ = oracle_sample_rate(inp, k_top, rows)
        total_pairs += sum(r + 1 for r in rows)
        total_sec += sec
    value = total_pairs / total_sec / 1e9
    sample = f"{n_rows} evenly spaced whole rows of the L={L} workload per step (all s <= t), {args.steps} steps"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": 1e3 * total_sec / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": workload_name(args.workload, c)},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def median_event_ms(pairs):
    return statistics.median(a.elapsed_time(b) for a, b in pairs)


def time_cfg1(idxc, synth, dev, reps=200):
    """Config 1 (L = 2048, H_I = 16, d_I = 64, k = 256): one idxc_indexer_prefill call writing scores and indices.
    About 3 us of roofline work: the call is bound by launch latency and by the ramp of two kernels, so the figure
    to report is microseconds per call. Inputs and outputs (21 MB) stay in L2 between repeats, as they would in a
    model that runs this shape."""
    c = synth.CONFIGS["cfg1"]
    L, H, d, k_top = c["L"], c["H"], c["d"], c["k_top"]
    inp = synth.prefill_inputs(L, H, d, seed=c["seed"], device=dev)
    scores = torch.empty((L, L), dtype=torch.float32, device=dev)
    topk = torch.empty((L, k_top), dtype=torch.int32, device=dev)

    def call():
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, scores_out=scores, topk_out=topk)
    for _ in range(10):
        call()
    evs = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        call()
        b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    idxc.poll_device_status()
    us = median_event_ms(evs) * 1e3
    # back to back, no events in between: the launch gaps overlap with the kernels
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(reps):
        call()
    b.record()
    torch.cuda.synchronize()
    us_stream = a.elapsed_time(b) * 1e3 / reps
    pairs = causal_pairs(L)
    us_graph = graph_replay_us(lambda i: call(), 50)
    idxc.poll_device_status()
    return {"workload": workload_name("cfg1", c) + ", scores + indices", "us_per_call": us, "us_per_call_back_to_back": us_stream,
            "us_per_call_graph": us_graph,
            "gpairs_per_s": pairs / (us_stream * 1e-6) / 1e9, "kernels_per_call": 2,
            "note": "latency-bound: 4.3 GFLOP and 10 MB of output per call are about 3 us of roofline work"}


def graph_replay_us(step, n_steps, reps=7):
    """n_steps calls step(0), step(1), ... captured ONCE into a CUDA graph on a side stream and replayed: microseconds per
    step of the median replay. The library's calls allocate nothing, never synchronise and only enqueue kernels on the
    caller's stream, so a serving loop can capture its decode step this way; the replay removes the host's launch cost and
    most of the launch-to-launch gap between the step's kernels."""
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    g = torch.cuda.CUDAGraph()
    try:
        with torch.cuda.stream(side):
            step(0)
            with torch.cuda.graph(g, stream=side):
                for i in range(n_steps):
                    step(i)
    except Exception as e:        # an auxiliary figure: a capture that fails must not take the bench line with it
        sys.stderr.write(f"graph capture failed, figure left out: {e}\n")
        torch.cuda.synchronize()
        return None
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    g.replay()
    torch.cuda.synchronize()
    ts = []
    for _ in range(reps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b) * 1e3 / n_steps)
    del g
    return statistics.median(ts)


def time_decode(idxc, synth, dev, peaks, steps, warmup):
    c = synth.CONFIGS["cfg3"]
    x = synth.decode_inputs(c["B"], c["H"], c["d"], c["len_lo"], c["len_hi"], seed=c["seed"], device=dev)
    B, k_top = c["B"], c["k_top"]
    topk = torch.empty((B, k_top), dtype=torch.int32, device=dev)
    ws = idxc.alloc_workspace(idxc.decode_workspace_bytes(B, x.max_len, c["H"], c["d"], k_top), dev)
    ld = (x.max_len + 31) // 32 * 32
    scores = ws[: B * ld * 4].view(torch.float32).view(B, ld)
    # the step as a caller runs it: ONE call (scores to the workspace, then top-k); then the scorer alone for its
    # roofline line
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(2 * steps)]
    for i in range(warmup + steps):
        j = i - warmup
        if j >= 0:
            ev[2 * j].record()
        idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, topk_out=topk, workspace=ws)
        if j >= 0:
            ev[2 * j + 1].record()
    torch.cuda.synchronize()
    idxc.poll_device_status()
    t_total = [ev[2 * j].elapsed_time(ev[2 * j + 1]) * 1e3 for j in range(steps)]
    for i in range(warmup + steps):
        j = i - warmup
        if j >= 0:
            ev[2 * j].record()
        idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top, scores_out=scores)
        if j >= 0:
            ev[2 * j + 1].record()
    torch.cuda.synchronize()
    t_score = [ev[2 * j].elapsed_time(ev[2 * j + 1]) * 1e3 for j in range(steps)]
    keys = int(x.lens.sum().item())
    bytes_k = keys * c["d"] * 2
    us_score, us_total = statistics.median(t_score), statistics.median(t_total)
    us_graph = graph_replay_us(lambda i: idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, x.max_len, k_top,
                                                             topk_out=topk, workspace=ws), 16)
    idxc.poll_device_status()
    gbs = bytes_k / (us_score * 1e-6) / 1e9
    # the consumer of the step's indices: sparse attention of the B new tokens over their selected cache rows
    # (128 heads, 576/512-column latent rows in a cache with the same row offsets; few queries: rows split over CTAs)
    att = synth.attention_inputs(B, x.k_cache.shape[0], 128, 576, seed=c["seed"], device=dev)
    a_out = torch.empty((B, 128, 512), dtype=torch.bfloat16, device=dev)
    a_ws = idxc.alloc_workspace(idxc.lib().idxc_sparse_attention_workspace_bytes(B, k_top), dev)
    for _ in range(3):
        idxc.sparse_attention(att.q, att.kv, topk, 512, 1.0 / 24.0, kv_base=x.k_offsets, out=a_out, workspace=a_ws, want_lse=False)
    ea, eb = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ea.record()
    for _ in range(10):
        idxc.sparse_attention(att.q, att.kv, topk, 512, 1.0 / 24.0, kv_base=x.k_offsets, out=a_out, workspace=a_ws, want_lse=False)
    eb.record()
    torch.cuda.synchronize()
    idxc.poll_device_status()
    us_attn = ea.elapsed_time(eb) * 1e3 / 10
    us_attn_graph = graph_replay_us(lambda i: idxc.sparse_attention(att.q, att.kv, topk, 512, 1.0 / 24.0, kv_base=x.k_offsets, out=a_out,
                                                                    workspace=a_ws, want_lse=False), 10)
    idxc.poll_device_status()
    attn_tf = 2.0 * 128 * (576 + 512) * B * k_top / (us_attn * 1e-6) / 1e12
    return {
        "sparse_attention_after": {"us": us_attn, "us_graph": us_attn_graph, "tflops_useful": attn_tf, "frac_of_bf16_peak": attn_tf / peaks["bf16_tflops"],
                                   "gathered_bytes": B * k_top * (576 + 256) * 2,
                                   "note": "B queries x k_top selected rows; with 32 queries four CTAs share a query and a second kernel merges their results"},
        "workload": f"cfg3: decode B={B} H_I={c['H']} d_I={c['d']} k_top={k_top}, sum(lens)={keys}",
        "us_per_step": us_total, "us_scorer": us_score, "us_topk": us_total - us_score,
        "us_per_step_graph": us_graph,
        "timing": "us_per_step: one idxc_indexer_decode call; us_scorer: the scorer kernel alone (scores only); us_topk: the difference; "
                  "us_per_step_graph: 16 such calls captured once into a CUDA graph, per step of the median replay",
        "k_cache_bytes": bytes_k,
        "l2": "766 MB of keys per step exceed the 126 MB L2: every step streams them from HBM",
        "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                     "frac": gbs / peaks["hbm_gbs"], "traffic": dram_traffic("score_decode_tc_kernel", "cfg3"),
                     "algorithmic_bytes": bytes_k, "kernel": "score_decode_tc_kernel",
                     "of": peaks["source"], "frac_of_nominal": gbs / NOMINAL["hbm_gbs"]},
        "frac_step_vs_hbm": bytes_k / (us_total * 1e-6) / 1e9 / peaks["hbm_gbs"],
        "frac_step_vs_hbm_graph": bytes_k / (us_graph * 1e-6) / 1e9 / peaks["hbm_gbs"] if us_graph else None,
    }


def _structure_ok(topk, q_begin, k_top):
    """Whole-output check on the device: per row min(k, t + 1) strictly ascending indices in [0, t], then -1."""
    rows = topk.shape[0]
    t = torch.arange(q_begin, q_begin + rows, device=topk.device)
    col = torch.arange(k_top, device=topk.device)
    valid = col[None, :] < torch.clamp(t + 1, max=k_top)[:, None]
    ok = bool(((topk >= 0) == valid).all()) and bool((topk[~valid] == -1).all())
    ok = ok and bool((torch.where(valid, topk, torch.zeros_like(topk)) <= t[:, None].to(topk.dtype)).all())
    d = topk[:, 1:] - topk[:, :-1]
    return ok and bool((d[valid[:, 1:]] > 0).all())


def time_schedule(idxc, synth, dev, L, H, d, k_top, n_layers, every, seed, reps, check_rows=4):
    """Config 4: the 1-in-`every` Full pattern against all-Full on the same independent per-layer inputs, and checks of the
    scheduled pass: every Shared layer returns its Full layer's buffer, every Full layer's output has the right structure
    and agrees with the oracle on sampled whole rows."""
    import oracle
    from tests.util import RTOL_BF16, assert_topk_valid, codes, f32
    layers = [synth.prefill_inputs(L, H, d, seed=seed, device=dev, layer=l) for l in range(n_layers)]
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H, d, k_top), dev)
    bufs = [torch.empty((L, k_top), dtype=torch.int32, device=dev) for _ in range(n_layers)]

    def run(pattern, keep=None):
        sch = idxc.Schedule(pattern)
        times = []
        for _ in range(reps + 1):
            sch.begin_pass()
            outs = []
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for l, ch in enumerate(pattern):
                x = layers[l]
                if ch == "F":
                    outs.append(sch.prefill_layer(l, x.q, x.k, x.w, k_top, topk_buf=bufs[l], workspace=ws))
                else:
                    outs.append(sch.prefill_layer(l, k_top=k_top, q_len=L))
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        calls = sch.stats()[2]
        if keep is not None:
            keep["outs"], keep["src"] = outs, [sch.source(l) for l in range(len(pattern))]
        sch.close()
        return statistics.median(times[1:]), calls // (reps + 1)

    pat = synth.uniform_pattern(n_layers, every)
    kept = {}
    t_sched, calls_sched = run(pat, kept)
    idxc.poll_device_status()
    # checks on the scheduled pass (outside the timed region)
    outs, src = kept["outs"], kept["src"]
    alias_ok = all(outs[l].data_ptr() == outs[src[l]].data_ptr() for l in range(n_layers))
    full_layers = [l for l, ch in enumerate(pat) if ch == "F"]
    structure_ok = all(_structure_ok(outs[l], 0, k_top) for l in full_layers)
    distinct_ok = all(not torch.equal(outs[a][-64:], outs[b][-64:]) for a, b in zip(full_layers, full_layers[1:]))
    rows_valid = rows_exact = 0
    for l in full_layers:
        rows = sorted({k_top - 1, k_top, L // 2 + 17 * l, L - 1} | {int(r) for r in torch.randint(k_top, L, (max(check_rows - 4, 0),),
                                                                                                  generator=torch.Generator().manual_seed(l))})
        # whole rows, each evaluated by the oracle at its own position
        host = synth.PrefillInputs(layers[l].q[rows].cpu(), layers[l].k.cpu(), layers[l].w[rows].cpu(), None, None, False)
        kc = codes(host.k)
        for j, t in enumerate(rows):
            o_sc, _ = oracle.indexer_prefill(codes(host.q[j:j + 1]), kc, f32(host.w[j:j + 1]), k_top, oracle.BF16, None, None, q_begin=t)
            rows_exact += bool(assert_topk_valid(outs[l][t].cpu().numpy(), o_sc[0, : t + 1], k_top, RTOL_BF16, what=f"layer {l} row {t}"))
            rows_valid += 1
    t_full, calls_full = run("F" * n_layers)
    idxc.poll_device_status()
    pairs = causal_pairs(L)
    return {"workload": f"cfg4: N={n_layers} layers, L={L}, H_I={H}, d_I={d}, k_top={k_top}, F every {every}, independent q/k/w per layer, seed {seed}",
            "ms_scheduled": t_sched, "ms_all_full": t_full, "ratio": t_full / t_sched,
            "indexer_calls": [calls_sched, calls_full],
            "gpairs_per_s_full_layers": pairs * calls_full / (t_full * 1e-3) / 1e9,
            "checks": {"shared_layers_alias_their_full_layer": alias_ok, "full_layers_structure_ok": structure_ok,
                       "consecutive_full_layers_differ": distinct_ok,
                       "oracle_rows_within_tolerance": rows_valid, "oracle_rows_identical": rows_exact,
                       "full_layers_checked": len(full_layers)}}


def time_layer_loop(idxc, synth, dev, L, k_top, n_layers, every, seed):
    """Fig. 2(b) with its attention step: per layer, a Full layer runs indexer + top-k, a Shared layer reuses the cached
    indices, and every layer runs the sparse attention over them (128 heads, 576/512-column latent rows; the same
    synthetic q and kv serve all layers). Compares the 1-in-`every` pattern with all-Full."""
    H_i, d_i = 64, 128
    pin = synth.prefill_inputs(L, H_i, d_i, seed=seed, device=dev, clustered=True)
    att = synth.attention_inputs(L, L, 128, 576, seed=seed, device=dev)
    topk = torch.empty((L, k_top), dtype=torch.int32, device=dev)
    out = torch.empty((L, 128, 512), dtype=torch.bfloat16, device=dev)
    ws_i = idxc.alloc_workspace(idxc.prefill_workspace_bytes(L, L, H_i, d_i, k_top), dev)
    ws_a = idxc.alloc_workspace(idxc.lib().idxc_sparse_attention_workspace_bytes(L, k_top), dev)
    scale = 1.0 / math.sqrt(576)

    def run(pattern):
        sch = idxc.Schedule(pattern)
        sch.begin_pass()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for layer, c in enumerate(pattern):
            if c == "F":
                t = sch.prefill_layer(layer, pin.q, pin.k, pin.w, k_top, topk_buf=topk, workspace=ws_i)
            else:
                t = sch.prefill_layer(layer, k_top=k_top, q_len=L)
            idxc.sparse_attention(att.q, att.kv, t, 512, scale, out=out, workspace=ws_a, want_lse=False)
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b)

    sched, full = synth.uniform_pattern(n_layers, every), "F" * n_layers
    run(sched)
    t_sched, t_full = run(sched), run(full)
    idxc.poll_device_status()
    return {"workload": f"{n_layers} layers, L={L}, k_top={k_top}: indexer (F layers only) + sparse attention (every layer)",
            "ms_scheduled": t_sched, "ms_all_full": t_full, "ratio": t_full / t_sched,
            "note": "the paper's end-to-end figures (1.82x prefill at 200K) include an FP8 indexer and the rest of the model; context only"}


def measure_fp8_gemm_peak(dev):
    """A denominator for the FP8 lines only (MEASURED_PEAKS.json holds no FP8 figure): the library's e4m3 GEMM,
    8192^3, best of 10 by CUDA events. None if this torch build has no such GEMM. Not on any timed path."""
    try:
        n = 8192
        a = torch.randn(n, n, device=dev).to(torch.float8_e4m3fn)
        b = torch.randn(n, n, device=dev).to(torch.float8_e4m3fn).t()
        one = torch.tensor(1.0, device=dev)
        for _ in range(3):
            torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
            e1.record()
            torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        return 2.0 * n ** 3 / (best * 1e-3) / 1e12
    except Exception:
        return None


def time_tmem_readout(idxc, dev, accumulators_per_warp=4096):
    """The rate at which the prefill epilogue's loads (tcgen05.ld 16x256b.x4, 8 warps per SM) read fp32 accumulators out
    of tensor memory when nothing else runs on the SM: the second roofline of the FP8 scorer. Measured live by the
    library's own measurement kernel."""
    for _ in range(2):
        nbytes = idxc.selftest_tmem_readout(accumulators_per_warp)
    evs = []
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        nbytes = idxc.selftest_tmem_readout(accumulators_per_warp)
        b.record()
        evs.append((a, b))
    torch.cuda.synchronize()
    idxc.poll_device_status()
    ms = min(a.elapsed_time(b) for a, b in evs)
    out = {"bytes_per_launch": nbytes, "ms": ms, "tbytes_per_s": nbytes / (ms * 1e-3) / 1e12,
           "what": "fp32 accumulator bytes read out of tensor memory per second over all SMs, the scorer's load pattern alone"}
    # the same loads while a ninth warp keeps the tensor pipe filling the two accumulators with the scorer's MMAs
    counters = torch.zeros(2, dtype=torch.int64, device=dev)
    for name, fp8 in (("under_fp8_mma", True), ("under_bf16_mma", False)):
        best = None
        for _ in range(4):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            nb = idxc.selftest_tmem_readout_under_mma(accumulators_per_warp, fp8, counters)
            b.record()
            torch.cuda.synchronize()
            t = a.elapsed_time(b)
            if best is None or t < best[0]:
                best = (t, int(counters[0].item()), int(counters[1].item()))
        idxc.poll_device_status()
        t, fills, cycles = best
        out[name] = {"ms": t, "tbytes_per_s": nb / (t * 1e-3) / 1e12, "accumulator_fills": fills,
                     "mma_tflops": fills * 2.0 * 128 * 256 * 128 / (t * 1e-3) / 1e12,
                     "reader_cycles_per_accumulator": cycles / accumulators_per_warp}
    # what one scheduler takes per warp instruction of the kinds the epilogue and the select are made of
    out["issue_cycles_per_warp_instruction"] = idxc.selftest_issue_rates(4096)
    out["under_mma_note"] = ("readers and MMAs run unordered beside each other on every SM; mma_tflops counts the fills completed while the "
                             "readers ran (2 x 128 x 256 x 128 flops each) over the launch time")
    return out


def time_decode_fp8(idxc, synth, dev, peaks, L, H, d, k_top, seed, decode_B, first_k=None, first_k_scale=None):
    """Decode step (one idxc_indexer_decode call: scorer + select) at batch decode_B on e4m3 caches of length L, timed on
    two cache sets used in turn so that no step finds its keys in L2. first_k / first_k_scale: keys of a prefill that
    become sequence 0 of set 0."""
    sets = []
    for si in range(2):
        x = synth.decode_inputs(decode_B, H, d, L, L, seed=seed, device=dev, layer=1 + si, fp8=True, lens=[L] * decode_B)
        if si == 0 and first_k is not None:
            x.k_cache[:L] = first_k
            x.k_scale[:L] = first_k_scale
        sets.append(x)
    dtop = torch.empty((decode_B, k_top), dtype=torch.int32, device=dev)
    dws = idxc.alloc_workspace(idxc.decode_workspace_bytes(decode_B, L, H, d, k_top, idxc.FP8_E4M3), dev)
    dld = (L + 31) // 32 * 32
    dscores = dws[: decode_B * dld * 4].view(torch.float32).view(decode_B, dld)
    ev_step, ev_score = [], []
    # The calls are enqueued behind a 10 ms spin kernel, so that all of them are queued before the first one runs: a step
    # of 50 us is otherwise as long as the host needs to issue it, and the events would time the host
    torch.cuda.synchronize()
    torch.cuda._sleep(20_000_000)
    for i in range(26):                                 # enqueued back to back: no host round trip inside a timed interval
        x = sets[i & 1]
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, L, k_top, x.q_scale, x.k_scale, topk_out=dtop, workspace=dws)
        b.record()
        ev_step.append((a, b))
    torch.cuda.synchronize()
    torch.cuda._sleep(20_000_000)
    for i in range(26):
        x = sets[i & 1]
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, L, k_top, x.q_scale, x.k_scale, scores_out=dscores)
        b.record()
        ev_score.append((a, b))
    torch.cuda.synchronize()
    idxc.poll_device_status()
    us = median_event_ms(ev_step[6:]) * 1e3
    us_sc = median_event_ms(ev_score[6:]) * 1e3
    nbytes = decode_B * L * (d + 4)

    def graph_step(i):
        x = sets[i & 1]
        idxc.indexer_decode(x.q_step, x.k_cache, x.w, x.k_offsets, x.lens, L, k_top, x.q_scale, x.k_scale, topk_out=dtop, workspace=dws)
    us_graph = graph_replay_us(graph_step, 24)          # the same alternation of the two cache sets, captured once
    idxc.poll_device_status()
    return {"B": decode_B, "us_per_step": us, "us_scorer": us_sc, "us_topk": us - us_sc, "bytes": nbytes,
            "us_per_step_graph": us_graph, "frac_of_hbm_graph": nbytes / (us_graph * 1e-6) / 1e9 / peaks["hbm_gbs"] if us_graph else None,
            "graph": "24 calls captured once into a CUDA graph, per step of the median replay",
            "frac_of_hbm": nbytes / (us * 1e-6) / 1e9 / peaks["hbm_gbs"],
            "scorer_frac_of_hbm": nbytes / (us_sc * 1e-6) / 1e9 / peaks["hbm_gbs"],
            "l2": f"two cache sets of {nbytes >> 20} MiB alternate between steps ({2 * nbytes >> 20} MiB > 126 MB L2): every step streams its keys from HBM"}


def time_fp8_chunked(idxc, synth, dev, peaks, L, chunk, H, d, k_top, seed, decode_B, n_layers, every, readout):
    """Config 5: FP8 (e4m3 + per-token scales) chunked prefill, query chunks of `chunk` rows against the full causal K:
    one Full layer (with the two kernels timed apart), the N-layer 1-in-`every` schedule against all-Full, then one
    decode step at batch `decode_B` on caches of length L, timed on two cache sets used in turn so that no step finds
    its keys in L2."""
    n_full = len([l for l in range(n_layers) if l % every == 0])
    layers = [synth.prefill_inputs(L, H, d, seed=seed, device=dev, fp8=True, layer=l) for l in range(n_full)]
    inp = layers[0]
    # the decode step (a 50 us pair of kernels whose time follows the SM clock) is timed first, before the seconds of
    # power-capped prefill below pull the clocks down; sequence 0 of set 0 holds the prefill's keys; two cache sets alternate
    decode = time_decode_fp8(idxc, synth, dev, peaks, L, H, d, k_top, seed, decode_B, inp.k, inp.k_scale)
    decode["order"] = "timed at the start of this section (the section's clock record covers the prefill that follows as well)"
    torch.cuda.empty_cache()
    topk = torch.empty((L, k_top), dtype=torch.int32, device=dev)
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(chunk, L, H, d, k_top, idxc.FP8_E4M3), dev)
    ld = (L + 31) // 32 * 32
    scores = ws[: chunk * ld * 4].view(torch.float32).view(chunk, ld)

    def layer(x, split, out):
        evs = []
        for q0 in range(0, L, chunk):
            sl = slice(q0, q0 + chunk)
            if split:
                e = [torch.cuda.Event(enable_timing=True) for _ in range(3)]
                e[0].record()
                idxc.indexer_prefill(x.q[sl], x.k, x.w[sl], k_top, x.q_scale[sl], x.k_scale, q_begin=q0, scores_out=scores)
                e[1].record()
                idxc.topk_rows(scores, k_top, out[sl], first_len=q0 + 1, len_step=1)
                e[2].record()
                evs.append(e)
            else:
                idxc.indexer_prefill(x.q[sl], x.k, x.w[sl], k_top, x.q_scale[sl], x.k_scale, q_begin=q0, topk_out=out[sl], workspace=ws)
        return evs

    layer(inp, False, topk)                             # warm-up
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    layer(inp, False, topk)
    e1.record()
    torch.cuda.synchronize()
    ms_layer = e0.elapsed_time(e1)
    evs = layer(inp, True, topk)
    torch.cuda.synchronize()
    t_sc = sum(e[0].elapsed_time(e[1]) for e in evs)
    t_tk = sum(e[1].elapsed_time(e[2]) for e in evs)
    idxc.poll_device_status()
    structure_ok = _structure_ok(topk, 0, k_top)
    pairs = causal_pairs(L)
    flops = 2.0 * H * d * pairs
    tf = flops / (t_sc * 1e-3) / 1e12
    acc_bytes = 4.0 * H * pairs                         # every (query, head, key) product is one fp32 accumulator element
    out = {"workload": f"cfg5: L={L} in {L // chunk} chunks of {chunk}, e4m3 + per-token scales, H_I={H}, d_I={d}, k_top={k_top}, seed {seed}",
           "ms_per_layer": ms_layer, "gpairs_per_s": pairs / (ms_layer * 1e-3) / 1e9,
           "ms_scorer": t_sc, "ms_topk": t_tk, "structure_ok": structure_ok,
           "roofline_tensor": {"bound": "tensor", "achieved": tf, "peak": 2 * peaks["bf16_tflops"], "unit": "TFLOP/s",
                               "frac": tf / (2 * peaks["bf16_tflops"]), "of": "2 x " + peaks["source"] + " bf16 burst peak (nominal FP8 : BF16 ratio; no FP8 figure is recorded for this box)",
                               "frac_of_sustained": tf / (2 * peaks["bf16_tflops_sustained"]),
                               "sustained_note": "a layer is 16 scorer launches of 1 to 10 ms back to back under the board's power cap "
                                                 "(see this section's clocks): the sustained bf16 figure is the like-for-like denominator",
                               "frac_of_nominal": tf / NOMINAL["fp8_tflops"], "kernel": "score_prefill_tc_kernel<fp8>"},
           "topk_kernel": {"ms_per_layer": t_tk, "achieved": (4.0 * pairs + 4.0 * L * k_top) / (t_tk * 1e-3) / 1e9, "unit": "GB/s",
                           "frac": (4.0 * pairs + 4.0 * L * k_top) / (t_tk * 1e-3) / 1e9 / peaks["hbm_gbs"]}}
    if readout:
        ach = acc_bytes / (t_sc * 1e-3) / 1e12
        out["roofline_readout"] = {"bound": "alu", "achieved": ach, "peak": readout["tbytes_per_s"], "unit": "TB/s of fp32 accumulator read out of tensor memory",
                                   "frac": ach / readout["tbytes_per_s"],
                                   "derivation": f"4 B x H_I = {4 * H} accumulator bytes per causal pair, {acc_bytes:.3e} B per layer, / scorer time; "
                                                 "peak = the same loads alone, measured in this run (tmem_readout section)"}
        if "under_fp8_mma" in readout:
            out["roofline_readout"]["peak_under_fp8_mma"] = readout["under_fp8_mma"]["tbytes_per_s"]
            out["roofline_readout"]["frac_under_fp8_mma"] = ach / readout["under_fp8_mma"]["tbytes_per_s"]
    # the gate: one min/max instruction per accumulator element on a pipe that issues 16 lanes per clock and scheduler
    # (measured: a warp's FMNMX every 2.0 cycles per scheduler), 4 schedulers per SM, at the SM clock's maximum
    props = torch.cuda.get_device_properties(dev)
    fmnmx_cycles = (readout or {}).get("issue_cycles_per_warp_instruction", {}).get("fmnmx", 2.0)     # measured in this run
    gate_peak = props.multi_processor_count * 4 * (32.0 / fmnmx_cycles) * (NOMINAL["sm_max_mhz"] * 1e6) / 1e12   # T elements / s
    gate_ach = acc_bytes / 4 / (t_sc * 1e-3) / 1e12
    out["roofline_gate"] = {"bound": "alu", "achieved": gate_ach, "peak": gate_peak, "unit": "T accumulator elements gated per second",
                            "frac": gate_ach / gate_peak,
                            "derivation": f"ReLU = one min/max per accumulator element; a scheduler takes one such warp instruction every {fmnmx_cycles:.2f} cycles "
                                          "(measured in this run, tmem_readout.issue_cycles_per_warp_instruction): "
                                          f"{props.multi_processor_count} SMs x 4 schedulers x 32 lanes / {fmnmx_cycles:.2f} x {NOMINAL['sm_max_mhz']} MHz; with e4m3 inputs this equals the tensor time "
                                          "of the accumulator (512 cycles per 128 x 256), and the epilogue's selects, compares and address arithmetic share the pipe"}
    fp8_peak = measure_fp8_gemm_peak(dev)
    if fp8_peak:
        out["fp8_gemm_peak_measured_here_tflops"] = fp8_peak
        out["scorer_frac_of_fp8_gemm_peak_measured_here"] = tf / fp8_peak
    # ---- the N-layer schedule: Full layers every `every`, against all-Full (which reuses the Full layers' inputs in turn:
    # the time of a layer does not depend on its values)
    bufs = [torch.empty((L, k_top), dtype=torch.int32, device=dev) for _ in range(2)]

    def run(pattern):
        sch = idxc.Schedule(pattern)
        sch.begin_pass()
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        n_f = 0
        for l, ch in enumerate(pattern):
            if ch == "F":
                x = layers[n_f % n_full]
                buf = bufs[n_f & 1]
                for q0 in range(0, L, chunk):
                    sl = slice(q0, q0 + chunk)
                    idxc.indexer_prefill(x.q[sl], x.k, x.w[sl], k_top, x.q_scale[sl], x.k_scale, q_begin=q0, topk_out=buf[sl], workspace=ws)
                n_f += 1
            # a Shared layer reuses the cached tensor: nothing is launched
        b.record()
        torch.cuda.synchronize()
        return a.elapsed_time(b), n_f

    pat = synth.uniform_pattern(n_layers, every)
    t_sched, f_sched = run(pat)
    t_full, f_full = run("F" * n_layers)
    idxc.poll_device_status()
    out["schedule"] = {"layers": n_layers, "ms_scheduled": t_sched, "ms_all_full": t_full, "ratio": t_full / t_sched,
                       "indexer_layers": [f_sched, f_full],
                       "note": "chunked calls per Full layer; Shared layers launch nothing (the schedule object's bookkeeping is host logic, timed in cfg4)"}
    del layers[1:]
    torch.cuda.empty_cache()
    out["decode"] = decode
    return out


def time_stream_topk(idxc, synth, dev, L, H, d, k_top, seed, fp8=False, q_begin=0, q_len=0):
    """Config 2 with the streaming top-k (IDXC_FLAG_STREAM_TOPK: the scorer's epilogue keeps per-row candidate lists instead
    of writing the scores) next to the ordinary step, calls interleaved; the index tensors must be identical.
    fp8 / q_begin / q_len: the same comparison on one query chunk [q_begin, q_begin + q_len) of an e4m3 prefill (config 5's
    shape: long rows)."""
    inp = synth.prefill_inputs(L, H, d, seed=seed, device=dev, clustered=not fp8, fp8=fp8)
    F = idxc.FLAG_STREAM_TOPK
    dt = idxc.FP8_E4M3 if fp8 else idxc.BF16
    q_len = q_len or L - q_begin
    sl = slice(q_begin, q_begin + q_len)
    q, w = inp.q[sl], inp.w[sl]
    qs = inp.q_scale[sl] if fp8 else None
    ws0 = idxc.alloc_workspace(idxc.prefill_workspace_bytes(q_len, L, H, d, k_top, dt), dev)
    ws1 = idxc.alloc_workspace(idxc.prefill_workspace_bytes(q_len, L, H, d, k_top, dt, F), dev)
    t0 = torch.empty((q_len, k_top), dtype=torch.int32, device=dev)
    t1 = torch.empty((q_len, k_top), dtype=torch.int32, device=dev)
    f0 = lambda: idxc.indexer_prefill(q, inp.k, w, k_top, qs, inp.k_scale, q_begin=q_begin, topk_out=t0, workspace=ws0)
    f1 = lambda: idxc.indexer_prefill(q, inp.k, w, k_top, qs, inp.k_scale, q_begin=q_begin, topk_out=t1, workspace=ws1, flags=F)
    for _ in range(2):
        f0(); f1()
    torch.cuda.synchronize()
    idxc.poll_device_status()
    ta, tb = [], []
    for _ in range(5):
        for f, acc in ((f0, ta), (f1, tb)):
            a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            a.record()
            for _ in range(2):
                f()
            b.record()
            torch.cuda.synchronize()
            acc.append(a.elapsed_time(b) / 2)
    idxc.poll_device_status()
    pairs = sum(range(q_begin + 1, q_begin + q_len + 1))
    ms0, ms1 = statistics.median(ta), statistics.median(tb)
    return {"workload": f"L={L}, rows {q_begin}..{q_begin + q_len - 1}, H_I={H}, d_I={d}, k_top={k_top}, {'e4m3' if fp8 else 'bf16, clustered keys'}, seed {seed}",
            "ms_ordinary": ms0, "ms_streaming": ms1, "gpairs_per_s_streaming": pairs / (ms1 * 1e-3) / 1e9,
            "indices_identical": bool(torch.equal(t0, t1)),
            "launches_per_call": {"ordinary": 2, "streaming": 4},
            "note": "streaming = scorer with per-row candidate lists + list select + the two ordinary kernels restricted to flagged rows; "
                    "the ordinary step is the default because the scorer's epilogue is the pace-setter and every per-score operation added to it costs more than the select saves"}


def time_quantize(idxc, dev, peaks, n_tokens, H, d):
    """Per-token bf16 -> e4m3 quantiser on query-shaped rows [n_tokens, H*d] and key-shaped rows [16 * n_tokens, d]
    (both larger than L2). Algorithmic bytes: 2 read + 1 written per element + 4 per token."""
    out = {}
    for name, rows, row_elems in (("queries", n_tokens, H * d), ("keys", 16 * n_tokens, d)):
        x = torch.randn((rows, row_elems), device=dev, dtype=torch.float32).to(torch.bfloat16)
        codes_out = torch.empty((rows, row_elems), dtype=torch.uint8, device=dev)
        scale_out = torch.empty((rows,), dtype=torch.float32, device=dev)
        for _ in range(3):
            idxc.quantize_e4m3(x, codes_out, scale_out)
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        for _ in range(10):
            idxc.quantize_e4m3(x, codes_out, scale_out)
        b.record()
        torch.cuda.synchronize()
        ms = a.elapsed_time(b) / 10
        nbytes = rows * row_elems * 3 + rows * 4
        gbs = nbytes / (ms * 1e-3) / 1e9
        out[name] = {"rows": rows, "row_elems": row_elems, "ms": ms, "bytes": nbytes,
                     "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                                  "frac": gbs / peaks["hbm_gbs"], "of": peaks["source"]}}
        del x, codes_out, scale_out
    return out


def time_overlap(idxc, dev, peaks, rows, k_top, n_layers):
    """Pairwise top-k index overlap (Appendix A) over n_layers index tensors [rows, k_top] in one launch, through the
    C-ABI call with the pointer and pair tables already on the device (the binding's own uploads of those tables are
    argument marshalling, not the kernel). Algorithmic bytes: each pair reads both tensors once (2 * rows * k_top * 4)."""
    import ctypes
    g = torch.Generator(device=dev).manual_seed(11)
    tops = []
    for l in range(n_layers):       # sorted random subsets of [0, 8 * k_top): valid ascending index rows
        t = torch.rand((rows, 8 * k_top), generator=g, device=dev).topk(k_top, dim=1).indices.to(torch.int32)
        tops.append(torch.sort(t, dim=1).values.contiguous())
    pairs = [(a, b) for a in range(n_layers) for b in range(a + 1, n_layers)]
    ptrs = torch.tensor([t.data_ptr() for t in tops], dtype=torch.int64, device=dev)
    pr = torch.tensor(pairs, dtype=torch.int32, device=dev).reshape(-1)
    means = torch.empty((len(pairs),), dtype=torch.float64, device=dev)
    L_ = idxc.lib()
    stream = ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)

    def call():
        st = L_.idxc_topk_overlap(ctypes.c_void_p(ptrs.data_ptr()), ctypes.c_void_p(pr.data_ptr()), len(pairs), rows, k_top,
                                  ctypes.c_void_p(means.data_ptr()), None, stream)
        assert st == 0
    call()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(5):
        call()
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / 5
    nbytes = len(pairs) * 2 * rows * k_top * 4
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"layers": n_layers, "pairs": len(pairs), "rows": rows, "k_top": k_top, "ms": ms, "mean_overlap": float(means.mean()),
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                         "of": peaks["source"], "note": "every tensor is read n_layers-1 times; the index tensors (403 MB) exceed L2"}}


def time_distill(idxc, dev, peaks, L, n_targets):
    """Forward value of the multi-layer distillation loss (Eq. 1) on causal rows of length t+1.
    Algorithmic bytes: 4 * (1 + n_targets) per causal pair."""
    g = torch.Generator(device=dev).manual_seed(13)
    scores = torch.randn((L, L), generator=g, device=dev)
    targets = []
    for _ in range(n_targets):
        p = torch.rand((L, L), generator=g, device=dev).tril_()
        p /= p.sum(dim=1, keepdim=True)
        targets.append(p)
    idxc.distill_kl(scores, targets)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(5):
        loss = idxc.distill_kl(scores, targets)
    b.record()
    torch.cuda.synchronize()
    ms = a.elapsed_time(b) / 5
    nbytes = causal_pairs(L) * 4 * (1 + n_targets)
    gbs = nbytes / (ms * 1e-3) / 1e9
    return {"rows": L, "targets": n_targets, "ms": ms, "loss": float(loss.item()),
            "roofline": {"bound": "hbm", "achieved": gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s", "frac": gbs / peaks["hbm_gbs"],
                         "of": peaks["source"]}}


def time_sparse_attention(idxc, synth, dev, peaks, L, n_q, k_top, seed, steps=3):
    """The consumer of the indices (Sec. 2.1): attention of the last n_q queries of an L-token prefill over the
    k_top rows the indexer picked for them (the real chain: indexer scores -> top-k -> attention), 128 heads over a
    shared latent row of 576 columns whose leading 512 are the value. Useful work: 2 * H * (d_qk + d_v) flops per
    (query, selected row); the kernel also recomputes nothing (scores once, P V in two halves)."""
    H_a, d_qk, d_v, H_i, d_i = 128, 576, 512, 64, 128
    pin = synth.prefill_inputs(L, H_i, d_i, seed=seed, device=dev, clustered=True)
    q0 = L - n_q
    topk = torch.empty((n_q, k_top), dtype=torch.int32, device=dev)
    ws = idxc.alloc_workspace(idxc.prefill_workspace_bytes(n_q, L, H_i, d_i, k_top), dev)
    idxc.indexer_prefill(pin.q[q0:], pin.k, pin.w[q0:], k_top, q_begin=q0, topk_out=topk, workspace=ws)
    del pin, ws
    inp = synth.attention_inputs(n_q, L, H_a, d_qk, seed=seed, device=dev)
    out = torch.empty((n_q, H_a, d_v), dtype=torch.bfloat16, device=dev)
    ws = idxc.alloc_workspace(idxc.lib().idxc_sparse_attention_workspace_bytes(n_q, k_top), dev)
    scale = 1.0 / math.sqrt(d_qk)
    for _ in range(2):
        idxc.sparse_attention(inp.q, inp.kv, topk, d_v, scale, out=out, workspace=ws, want_lse=False)
    idxc.poll_device_status()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    for _ in range(steps):
        idxc.sparse_attention(inp.q, inp.kv, topk, d_v, scale, out=out, workspace=ws, want_lse=False)
    b.record()
    torch.cuda.synchronize()
    idxc.poll_device_status()
    ms = a.elapsed_time(b) / steps
    selected = int((topk >= 0).sum().item())
    flops = 2.0 * H_a * (d_qk + d_v) * selected
    tf = flops / (ms * 1e-3) / 1e12
    gather_bytes = selected * (d_qk + d_v // 2) * 2
    return {"workload": f"last {n_q} queries of an L={L} prefill, H=128, d_qk=576, d_v=512, k_top={k_top}, indices from the indexer",
            "ms": ms, "queries_per_s": n_q / (ms * 1e-3), "selected_rows": selected,
            "gathered_bytes": gather_bytes,
            "roofline": {"bound": "tensor", "achieved": tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
                         "frac": tf / peaks["bf16_tflops"], "of": peaks["source"] + " burst peak",
                         "frac_of_sustained": tf / peaks["bf16_tflops_sustained"], "frac_of_nominal": tf / NOMINAL["bf16_tflops"],
                         "traffic": dram_traffic("sparse_attn_kernel", f"L{L}_q{n_q}"),
                         "note": "the kernel draws the board's full power: inside a long run the clocks settle near 1.6 GHz "
                                 "(sw_power_cap) and the time is about 15-20 % above a cold run of this section alone"}}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=["cfg1", "cfg2"])
    ap.add_argument("--ref-rows", type=int, default=128, help="rows per step of the reference (oracle) arm")
    ap.add_argument("--cpu-rows", type=int, default=1024, help="rows of the cpu_baseline sample")
    ap.add_argument("--e2e-steps", type=int, default=32, help="steps of the end-to-end loop (its first copy-in and last copy-out are not overlapped: few steps overstate them)")
    ap.add_argument("--no-extras", action="store_true", help="only the headline workload (config 2)")
    ap.add_argument("--quick", action="store_true", help="extra sections at reduced sizes (config 4 with 8 layers of L=32768, config 5 at L=32768): for profiling runs, not for reported numbers")
    ap.add_argument("--full", action="store_true", help="accepted for compatibility: full sizes are the default")
    ap.add_argument("--L", type=int, default=0, help="override the workload's sequence length (small profiling cases)")
    ap.add_argument("--only-decode", action="store_true", help="run only the decode section (profiling)")
    ap.add_argument("--only-decode-fp8", action="store_true", help="run only the batch-8 e4m3 decode step of config 5 (profiling)")
    ap.add_argument("--only-stream-topk", action="store_true", help="run only the streaming top-k section (profiling; --L sets the length)")
    ap.add_argument("--stream-fp8-chunk", type=int, default=-1, help="with --only-stream-topk: compare on the config-5 query chunk that starts at this row (e4m3, L = 131072 unless --L is given)")
    ap.add_argument("--only-sparse-attention", action="store_true", help="run only the sparse-attention section (profiling)")
    ap.add_argument("--only-layer-loop", action="store_true", help="run only the indexer + attention layer loop section")
    ap.add_argument("--only-fp8", action="store_true", help="run only the FP8 chunked-prefill section (profiling; --L sets the length)")
    ap.add_argument("--only-tools", action="store_true", help="run only the distillation-loss, overlap and quantiser sections (profiling)")
    ap.add_argument("--sa-queries", type=int, default=8192, help="queries of the sparse-attention section")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3

    if args.impl == "reference":
        rank = int(os.environ.get("RANK", "0"))
        run_reference(args, rank)
        return

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the indexer has no CPU path (use --impl reference for the oracle)")
    from paper_2603_12201_b200 import dist as pdist
    _, _, local = pdist.env_rank_world()
    # IDXC_BENCH_BACKEND=gloo is a functional smoke path for boxes with fewer GPUs than ranks: the ranks then
    # share the visible GPUs and the (host-side) timing reduction goes through gloo. Numbers from it mean nothing.
    backend = os.environ.get("IDXC_BENCH_BACKEND", "nccl")
    dev = torch.device("cuda", local % torch.cuda.device_count() if backend == "gloo" else local)
    torch.cuda.set_device(dev)
    rank, world = pdist.init(backend, dev)
    barrier = pdist.barrier

    def max_over_ranks(x, w, device):
        return pdist.max_over_ranks(x, w, "cpu" if backend == "gloo" else device)
    from paper_2603_12201_b200 import binding as idxc
    from paper_2603_12201_b200 import synth
    idxc.lib()
    peaks = load_peaks()

    def section(fn, *a, **kw):
        """Runs one section with the clock sampler around it; the section's dict gets a `clocks` entry. A section that
        raises is reported as {"error": ...} (and on stderr) instead of taking the headline line with it."""
        with ClockSampler(local) as clk:
            try:
                res = fn(*a, **kw)
                torch.cuda.synchronize()
            except Exception as e:
                import traceback
                traceback.print_exc()
                res = {"error": f"{type(e).__name__}: {e}"[:400]}
        res["clocks"] = clk.summary()
        torch.cuda.empty_cache()
        return res

    c5 = synth.CONFIGS["cfg5"]
    if args.only_decode:
        print(json.dumps({"decode": section(time_decode, idxc, synth, dev, peaks, steps=max(args.steps, 1), warmup=args.warmup)}),
              flush=True)
        return
    if args.only_decode_fp8:
        print(json.dumps({"decode_fp8": section(time_decode_fp8, idxc, synth, dev, peaks, args.L or c5["L"], c5["H"], c5["d"], c5["k_top"],
                                                c5["seed"], c5["decode_B"])}), flush=True)
        return
    if args.only_stream_topk:
        c2 = synth.CONFIGS["cfg2"]
        if args.stream_fp8_chunk >= 0:
            print(json.dumps({"stream_topk": section(time_stream_topk, idxc, synth, dev, args.L or c5["L"], c5["H"], c5["d"], c5["k_top"], c5["seed"],
                                                     fp8=True, q_begin=args.stream_fp8_chunk, q_len=c5["chunk"])}), flush=True)
        else:
            print(json.dumps({"stream_topk": section(time_stream_topk, idxc, synth, dev, args.L or c2["L"], c2["H"], c2["d"], c2["k_top"], c2["seed"])}), flush=True)
        return
    if args.only_layer_loop:
        print(json.dumps({"layer_loop": section(time_layer_loop, idxc, synth, dev, args.L or 32768, 2048, 4, 4, seed=8)}), flush=True)
        return
    if args.only_fp8:
        ro = section(time_tmem_readout, idxc, dev)
        L5 = args.L or c5["L"]
        print(json.dumps({"tmem_readout": ro,
                          "fp8_chunked": section(time_fp8_chunked, idxc, synth, dev, peaks, L5, min(c5["chunk"], L5), c5["H"], c5["d"],
                                                 c5["k_top"], c5["seed"], c5["decode_B"], 8 if args.quick else c5["N"], c5["every"], ro)}), flush=True)
        return
    if args.only_tools:
        print(json.dumps({"distill_kl": section(time_distill, idxc, dev, peaks, 16384, 2),
                          "topk_overlap": section(time_overlap, idxc, dev, peaks, 8192, c5["k_top"], 6),
                          "quantize_e4m3": section(time_quantize, idxc, dev, peaks, 32768, c5["H"], c5["d"])}), flush=True)
        return
    if args.only_sparse_attention:
        print(json.dumps({"sparse_attention": section(time_sparse_attention, idxc, synth, dev, peaks, args.L or 32768, args.sa_queries, 2048,
                                                      seed=7, steps=max(args.steps, 1))}), flush=True)
        return
    c = dict(synth.CONFIGS[args.workload])
    if args.L:
        c["L"] = args.L
    L, H, d, k_top = c["L"], c["H"], c["d"], c["k_top"]
    # independent problem per rank (weak scaling): same shape, rank-specific seed
    inp = synth.prefill_inputs(L, H, d, seed=pdist.rank_seed(c["seed"], rank), device=dev, fp8=c["fp8"], clustered=c["clustered"])
    ld = (L + 31) // 32 * 32
    scores = torch.empty((L, ld), dtype=torch.float32, device=dev)
    topk = torch.empty((L, k_top), dtype=torch.int32, device=dev)
    pairs = causal_pairs(L)
    K, W = args.steps, args.warmup

    def step(evs=None):
        # the two halves of idxc_indexer_prefill as two public calls, so that CUDA events can time each kernel
        if evs:
            evs[0].record()
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, inp.q_scale, inp.k_scale, scores_out=scores)   # scorer launch
        if evs:
            evs[1].record()
        idxc.topk_rows(scores, k_top, topk, first_len=1, len_step=1)                                    # top-k launch
        if evs:
            evs[2].record()

    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(3)] for _ in range(K)]
    with ClockSampler(local) as clk:                 # started before the warm-up: its first queries are slow and hold the interpreter
        for _ in range(W):
            step()
        torch.cuda.synchronize()
        barrier(world)
        launches0 = idxc.launch_count()
        clk.reset()
        t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        t_start.record()
        for i in range(K):
            step(evs[i])
        t_end.record()
        launches = idxc.launch_count() - launches0      # (the library counts a launch when it enqueues it)
        # The clock sampler keeps running over another 0.15 s of the same load behind the timed region (not timed: t_end is
        # already recorded): NVML reports a throttle reason up to a few hundred ms after the clocks have dropped, and a
        # region of K = 20 steps is over before that
        for _ in range(max(1, int(0.15 / 0.0072))):
            step()
        torch.cuda.synchronize()
    barrier(world)
    idxc.poll_device_status()
    total_ms = max_over_ranks(t_start.elapsed_time(t_end), world, dev)
    ms_per_step = total_ms / K
    value = pdist.whole_job_rate(pairs, K, total_ms, world) / 1e9
    scorer_ms = statistics.mean(e[0].elapsed_time(e[1]) for e in evs)
    topk_ms = statistics.mean(e[1].elapsed_time(e[2]) for e in evs)
    flops = 2.0 * H * d * pairs
    achieved_tf = flops / (scorer_ms * 1e-3) / 1e12
    topk_bytes = 4.0 * pairs + 4.0 * L * k_top
    topk_gbs = topk_bytes / (topk_ms * 1e-3) / 1e9
    case = f"L{L}" if args.workload == "cfg2" else f"{args.workload}_L{L}"
    roofline = {
        "bound": "tensor", "achieved": achieved_tf, "peak": peaks["bf16_tflops"], "unit": "TFLOP/s",
        "frac": achieved_tf / peaks["bf16_tflops"],
        "traffic": dram_traffic("score_prefill_tc_kernel", case),
        "algorithmic_bytes": inp.q.numel() * inp.q.element_size() + inp.k.numel() * inp.k.element_size() + inp.w.numel() * 4 + 4 * pairs,
        "kernel": "score_prefill_tc_kernel", "ms_per_launch": scorer_ms, "of": peaks["source"] + " burst peak",
        "frac_of_sustained": achieved_tf / peaks["bf16_tflops_sustained"],
        "frac_of_nominal": achieved_tf / NOMINAL["bf16_tflops"],
        "targets": "north star: prefill scoring >= 60 % of the dense BF16 peak, decode indexing >= 70 % of HBM bandwidth; judged here "
                   "on the fractions of the peaks MEASURED on this box (cuBLAS bf16 GEMM, copy bandwidth); frac_of_nominal gives the "
                   "same against the data-sheet figures (2250 TFLOP/s, 7.7 TB/s)",
        "algorithmic_flops_per_launch": flops,
        "topk_kernel": {"ms_per_launch": topk_ms, "launches": max(1, launches // K - 1),
                        "note": "one idxc_topk_rows call; a long prefill's rows are cut by length into up to three launches of "
                                "topk_rows_kernel instances, timed and counted together (traffic: their sum)",
                        "bound": "hbm", "achieved": topk_gbs, "peak": peaks["hbm_gbs"], "unit": "GB/s",
                        "frac": topk_gbs / peaks["hbm_gbs"], "frac_of_nominal": topk_gbs / NOMINAL["hbm_gbs"],
                        "algorithmic_bytes": topk_bytes, "traffic": dram_traffic("topk_rows_kernel", case)},
    }

    # ---- the same layer through the single user call (scores through the workspace), device-resident inputs
    ws_c = scores.view(torch.uint8).view(-1)
    for _ in range(2):
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, inp.q_scale, inp.k_scale, topk_out=topk, workspace=ws_c)
    c0, c1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    c0.record()
    for _ in range(K):
        idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, inp.q_scale, inp.k_scale, topk_out=topk, workspace=ws_c)
    c1.record()
    torch.cuda.synchronize()
    combined_ms = c0.elapsed_time(c1) / K

    # ---- the select by itself, after a pause in which the board leaves the power limit the scorer holds it at: the
    # select's time follows the SM clock (it is bound by instruction issue, not by bytes), so both figures are given
    # with the clock they were taken at
    time.sleep(0.5)
    with ClockSampler(local) as clk_alone:
        for _ in range(3):
            idxc.topk_rows(scores, k_top, topk, first_len=1, len_step=1)
        a0, a1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a0.record()
        for _ in range(20):
            idxc.topk_rows(scores, k_top, topk, first_len=1, len_step=1)
        a1.record()
        torch.cuda.synchronize()
    topk_alone_ms = a0.elapsed_time(a1) / 20
    alone_gbs = topk_bytes / (topk_alone_ms * 1e-3) / 1e9
    roofline["topk_kernel"]["alone"] = {"ms_per_launch": topk_alone_ms, "achieved": alone_gbs, "frac": alone_gbs / peaks["hbm_gbs"],
                                        "sm_mhz": clk_alone.summary()["sm_mhz"],
                                        "note": "20 calls back to back without the scorer between them; the figure above is taken inside the "
                                                "timed loop, at the clock the top-level `clocks` entry records"}

    # ---- e2e: host buffers; every step copies its inputs H2D (pinned) and its result D2H inside the timed
    # region. Steps are software-pipelined over three streams with double-buffered device inputs and outputs
    # (copy-in of step i+1 and copy-out of step i-1 overlap the kernels of step i), as a serving loop would.
    hq = torch.empty(inp.q.shape, dtype=inp.q.dtype, pin_memory=True).copy_(inp.q)
    hk = torch.empty(inp.k.shape, dtype=inp.k.dtype, pin_memory=True).copy_(inp.k)
    hw = torch.empty(inp.w.shape, dtype=inp.w.dtype, pin_memory=True).copy_(inp.w)
    hout = [torch.empty(topk.shape, dtype=topk.dtype, pin_memory=True) for _ in range(2)]
    dq = [torch.empty_like(inp.q) for _ in range(2)]
    dk = [torch.empty_like(inp.k) for _ in range(2)]
    dw = [torch.empty_like(inp.w) for _ in range(2)]
    dtop = [topk, torch.empty_like(topk)]
    ws = scores.view(torch.uint8).view(-1)
    s_in, s_run, s_out = torch.cuda.Stream(dev), torch.cuda.Stream(dev), torch.cuda.Stream(dev)

    def e2e_run(n_steps):
        in_done = [None, None]      # event: inputs of the step using buffer b have landed
        run_done = [None, None]     # event: kernels of the step using buffer b have finished
        out_done = [None, None]     # event: result of the step using buffer b has been copied out
        for i in range(n_steps):
            b = i & 1
            with torch.cuda.stream(s_in):
                if run_done[b] is not None:
                    s_in.wait_event(run_done[b])             # the kernels that read this input buffer are done
                dq[b].copy_(hq, non_blocking=True)
                dk[b].copy_(hk, non_blocking=True)
                dw[b].copy_(hw, non_blocking=True)
                in_done[b] = s_in.record_event()
            with torch.cuda.stream(s_run):
                s_run.wait_event(in_done[b])
                if out_done[b] is not None:
                    s_run.wait_event(out_done[b])            # the previous result in this buffer has left
                idxc.indexer_prefill(dq[b], dk[b], dw[b], k_top, topk_out=dtop[b], workspace=ws, stream=s_run)   # the user's call
                run_done[b] = s_run.record_event()
            with torch.cuda.stream(s_out):
                s_out.wait_event(run_done[b])
                hout[b].copy_(dtop[b], non_blocking=True)
                out_done[b] = s_out.record_event()
        for st in (s_in, s_run, s_out):
            torch.cuda.current_stream().wait_stream(st)

    torch.cuda.synchronize()
    e2e_run(2)
    torch.cuda.synchronize()
    barrier(world)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for st in (s_in, s_run, s_out):
        st.wait_event(e0)
    e2e_run(args.e2e_steps)
    e1.record()
    torch.cuda.synchronize()
    e2e_ms = max_over_ranks(e0.elapsed_time(e1), world, dev)
    h2d = sum(t.numel() * t.element_size() for t in (hq, hk, hw))
    d2h = hout[0].numel() * hout[0].element_size()
    e2e = {"value": pdist.whole_job_rate(pairs, args.e2e_steps, e2e_ms, world) / 1e9, "unit": UNIT, "h2d_bytes_per_step": h2d,
           "d2h_bytes_per_step": d2h, "ms_per_step": e2e_ms / args.e2e_steps, "steps": args.e2e_steps,
           "pipelined": "3 streams, double-buffered inputs and results"}
    ref_top = torch.empty_like(topk)
    idxc.indexer_prefill(inp.q, inp.k, inp.w, k_top, inp.q_scale, inp.k_scale, topk_out=ref_top, workspace=ws)
    torch.cuda.synchronize()
    assert torch.equal(hout[0].to(dev), ref_top) and torch.equal(hout[1].to(dev), ref_top)
    topk.copy_(ref_top)

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": K, "warmup": W,
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "fp8_e4m3" if c["fp8"] else "bf16", "data": "synthetic",
        "config": {"workload": workload_name(args.workload, c),
                   "parallelism": f"independent problem per GPU x{world}",
                   "l2": (f"inputs {(inp.q.numel() * inp.q.element_size()) >> 20} MiB and scores "
                          f"{scores.numel() * 4 >> 20} MiB per step exceed the 126 MB L2; no flush needed"
                          if inp.q.numel() * inp.q.element_size() + scores.numel() * 4 > (126 << 20) else
                          f"inputs {(inp.q.numel() * inp.q.element_size()) >> 20} MiB and scores {scores.numel() * 4 >> 20} MiB "
                          "fit the 126 MB L2: this small parity-size case is timed L2-warm (it is not the bench workload)")},
        "roofline": roofline, "e2e": e2e, "gpu_launches": launches,
        "clocks": dict(clk.summary(), window="the timed region and 0.15 s of the same load behind it (NVML shows a throttle reason late)"),
        "kernel_ms": {"scorer": scorer_ms, "topk": topk_ms, "combined_call": combined_ms},
    }

    if rank == 0 and world == 1:
        # ---- the oracle on this machine's host cores, bounded sample of the same workload; doubles as a parity spot check
        host = synth.PrefillInputs(inp.q.cpu(), inp.k.cpu(), inp.w.cpu(),
                                   None if inp.q_scale is None else inp.q_scale.cpu(),
                                   None if inp.k_scale is None else inp.k_scale.cpu(), inp.fp8)
        rows = sample_rows(L, args.cpu_rows)
        import oracle
        rate, sec, o_tk = oracle_sample_rate(host, k_top, rows)
        g_tk = topk[rows].cpu().numpy()
        same = sum(int((g_tk[j] == o_tk[j]).all()) for j in range(len(rows)))
        line["cpu_baseline"] = {
            "value": rate / 1e9, "unit": UNIT, "cores": oracle.threads(), "kind": "oracle",
            "sample": f"{len(rows)} evenly spaced whole rows (all s <= t) of the same inputs, {sec:.1f} s",
            "rows_with_identical_index_set": f"{same}/{len(rows)}"}
        if not args.no_extras:
            del hq, hk, hw, dq, dk, dw, dtop, hout, inp, host, scores, ws, ws_c
            torch.cuda.empty_cache()
            c4 = synth.CONFIGS["cfg4"]
            line["cfg1"] = section(time_cfg1, idxc, synth, dev)
            line["decode"] = section(time_decode, idxc, synth, dev, peaks, steps=max(K, 10), warmup=W)
            n_layers, sched_L = (8, 32768) if args.quick else (c4["N"], c4["L"])
            line["schedule"] = section(time_schedule, idxc, synth, dev, sched_L, c4["H"], c4["d"], c4["k_top"], n_layers, c4["every"],
                                       seed=c4["seed"], reps=1)
            line["sparse_attention"] = section(time_sparse_attention, idxc, synth, dev, peaks, 32768, args.sa_queries, c4["k_top"], seed=7)
            line["layer_loop"] = section(time_layer_loop, idxc, synth, dev, 32768, c4["k_top"], 4, c4["every"], seed=8)
            line["distill_kl"] = section(time_distill, idxc, dev, peaks, 16384, 2)
            line["topk_overlap"] = section(time_overlap, idxc, dev, peaks, 8192, c5["k_top"], 6)
            line["quantize_e4m3"] = section(time_quantize, idxc, dev, peaks, 32768, c5["H"], c5["d"])
            line["tmem_readout"] = section(time_tmem_readout, idxc, dev)
            fp8_L, fp8_layers = (32768, 8) if args.quick else (c5["L"], c5["N"])
            line["fp8_chunked"] = section(time_fp8_chunked, idxc, synth, dev, peaks, fp8_L, c5["chunk"], c5["H"], c5["d"], c5["k_top"],
                                          c5["seed"], c5["decode_B"], fp8_layers, c5["every"], line["tmem_readout"])
            c2 = synth.CONFIGS["cfg2"]
            line["stream_topk"] = section(time_stream_topk, idxc, synth, dev, c2["L"], c2["H"], c2["d"], c2["k_top"], c2["seed"])
            # the five workloads in one place, inside the roofline block and again at the very end of the line
            f8, dc, sc = line["fp8_chunked"], line["decode"], line["schedule"]
            def summarise():
                return {
                    "cfg1": {"us_per_call": line["cfg1"]["us_per_call"], "us_back_to_back": line["cfg1"]["us_per_call_back_to_back"],
                             "us_graph": line["cfg1"]["us_per_call_graph"]},
                    "cfg2": {"gpairs_per_s": value, "ms_per_step": ms_per_step, "scorer_frac_of_bf16_peak": roofline["frac"],
                             "topk_frac_of_hbm": roofline["topk_kernel"]["frac"],
                             "streaming_topk_ms": line["stream_topk"]["ms_streaming"], "streaming_topk_identical": line["stream_topk"]["indices_identical"]},
                    "cfg3": {"us_per_step": dc["us_per_step"], "scorer_frac_of_hbm": dc["roofline"]["frac"], "step_frac_of_hbm": dc["frac_step_vs_hbm"],
                             "us_per_step_graph": dc["us_per_step_graph"], "step_frac_of_hbm_graph": dc["frac_step_vs_hbm_graph"]},
                    "cfg4": {"workload": sc["workload"], "ms_scheduled": sc["ms_scheduled"], "ms_all_full": sc["ms_all_full"], "ratio": sc["ratio"],
                             "gpairs_per_s_full_layers": sc["gpairs_per_s_full_layers"], "checks": sc["checks"]},
                    "cfg5": {"workload": f8["workload"], "ms_per_full_layer": f8["ms_per_layer"], "gpairs_per_s": f8["gpairs_per_s"],
                             "scorer_frac_of_2x_bf16_peak": f8["roofline_tensor"]["frac"],
                             "scorer_frac_of_2x_bf16_sustained": f8["roofline_tensor"]["frac_of_sustained"],
                             "scorer_frac_of_tmem_readout": f8.get("roofline_readout", {}).get("frac"),
                             "scorer_frac_of_gate_rate": f8["roofline_gate"]["frac"],
                             "schedule_ratio": f8["schedule"]["ratio"], "decode_B8_us": f8["decode"]["us_per_step"],
                             "decode_frac_of_hbm": f8["decode"]["frac_of_hbm"], "decode_B8_us_graph": f8["decode"]["us_per_step_graph"],
                             "decode_frac_of_hbm_graph": f8["decode"]["frac_of_hbm_graph"]},
                }
            try:
                by_config = summarise()
            except (KeyError, TypeError) as e:      # a section reported an error instead of its figures
                by_config = {"error": f"summary incomplete: {type(e).__name__}: {e}"}
            line["roofline"]["by_config"] = by_config
            line["summary"] = by_config
    if rank == 0:
        print(json.dumps(line), flush=True)
    pdist.shutdown(world)


if __name__ == "__main__":
    main()
