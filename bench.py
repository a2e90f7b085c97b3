#!/usr/bin/env python
"""Benchmark of the Parallel Track (PT) forward pass on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2|cfg3|cfg1|cfg4|cfg0|cfg2_kv8|cfg4_kv8|pt30b_prefill|pt30b_decode]
                    [--extra cfg3,cfg1] [--impl ours|reference]

One JSON line on stdout.  A "step" is one pass of the whole hot path over one batch: one
decode step (cfg2, cfg4) or one prefill (cfg1, cfg3) through every layer and track-sync.
`value` is tokens/s with inputs resident in HBM; `e2e` is the same call made from pinned host
buffers with the host<->device copies inside the timed region.  With N > 1 (torchrun) every
rank runs the same workload on its own batch (weak scaling, no data-path collective: batch
rows are independent) and rank 0 reports the aggregate over the slowest rank.

`--impl reference` times the CPU oracle (float64 NumPy, as it stands) on a bounded sample of
the same workload on the host cores.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

from paper_2602_07306_b200 import inputs as I  # noqa: E402

# DRAM traffic of k_decode_attn_tma<128> from its ncu capture (profiles/decode_attn_tma_T8_B8_kv2049.md:
# 8 sequences instead of 64, same kernel): dram read + write bytes per launch over the algorithmic K/V
# bytes of that launch.  Traffic is proportional to the keys read, so a bench launch is scaled by its own
# algorithmic bytes.  The counters belong to one version of the kernel's source files: their SHA-256 is kept
# beside them, and when the files on disk differ the bench reports "traffic": null with the reason.
DECODE_ATTN_TRAFFIC_RATIO = (541.24e6 + 4.00e6) / 537.13e6
DECODE_ATTN_TRAFFIC_SOURCE = (("paper_2602_07306_b200/csrc/pt_tc_attn.cu", "paper_2602_07306_b200/csrc/pt_ptx.cuh"),
                              "58ea08e5b2a28ea033c2102a8313e6851f5d5a19e263cc48595495108d95f25c")


def decode_attn_traffic_ratio():
    """(ratio, None) while the kernel's sources are the ones the counters were taken on, else (None, reason)."""
    import hashlib
    paths, want = DECODE_ATTN_TRAFFIC_SOURCE
    h = hashlib.sha256()
    try:
        for path in paths:
            with open(os.path.join(ROOT, path), "rb") as f:
                h.update(f.read())
    except OSError as e:
        return None, f"kernel source not readable: {e}"
    if h.hexdigest() != want:
        return None, f"{' or '.join(paths)} changed since the ncu counters were taken"
    return DECODE_ATTN_TRAFFIC_RATIO, None

FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# ------------------------------------------------------------------------------ clocks

class ClockSampler:
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, dev):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thr = None
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                self.h = pynvml.nvmlDeviceGetHandleByUUID("GPU-" + str(torch.cuda.get_device_properties(dev).uuid))
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(dev.index or 0)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
        except Exception:
            self.nv = None

    def _loop(self):
        nv = self.nv
        names = {"hw_slowdown": 0x8, "sw_power_cap": 0x4, "sw_thermal_slowdown": 0x20,
                 "hw_thermal_slowdown": 0x40, "hw_power_brake": 0x80}
        while not self._stop.is_set():
            try:
                self.samples.append(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM))
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.h)
                for k, bit in names.items():
                    if r & bit:
                        self.reasons.add(k)
            except Exception:
                pass
            self._stop.wait(0.05)

    def __enter__(self):
        if self.nv:
            self._thr = threading.Thread(target=self._loop, daemon=True)
            self._thr.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thr:
            self._thr.join()

    def summary(self):
        med = float(np.median(self.samples)) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# ------------------------------------------------------------------------------ workloads

def kv8(wl):
    """Workloads whose name ends in _kv8 keep their cache in the E4M3 format (8-bit codes + one fp32 scale per vector)."""
    return wl.name.endswith("_kv8")


def algorithmic(wl, B, lens=None, S=None):
    """Algorithmic work of one step (no padding, no re-reads, causal triangle only)."""
    P = wl.params_per_track_layer()
    dh = wl.head_dim
    if wl.mode == "decode":
        keys = int(np.sum(np.asarray(lens, np.int64) + 1))
        vec_bytes = dh + 4 if kv8(wl) else dh * 2          # one cached vector: codes + scale, or bf16 values
        kv_read = wl.T * wl.L * 2 * wl.kv_heads * vec_bytes * keys
        kv_write = wl.T * wl.L * 2 * wl.kv_heads * vec_bytes * B
        weights = wl.T * wl.L * P * 2
        return {"bytes": kv_read + kv_write + weights, "kv_read_bytes": kv_read, "weight_bytes": weights,
                "attn_bytes_per_layer": kv_read // wl.L}
    tokens = B * S
    gemm = 2 * wl.T * wl.L * P * tokens
    attn = wl.T * wl.L * B * 4 * wl.heads * dh * S * (S + 1) // 2
    return {"flops": gemm + attn, "gemm_flops": gemm, "attn_flops": attn}


TRACK_PARALLEL = {"on": False, "world": 1, "rank": 0, "tracks": 0}


def make_model(wl, dev, max_pos):
    """With --parallel tracks `wl` is one rank's share (T / N tracks, the paper's placement) of a
    model of TRACK_PARALLEL["tracks"] tracks and the track-sync is one NCCL all-reduce per track
    block; otherwise every rank holds the whole model."""
    from paper_2602_07306_b200 import pt
    m = pt.Model(T=wl.T, D=wl.D, L=wl.L, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads, ffn=wl.ffn,
                 dtype=wl.dtype, rope_base=wl.rope_base, rms_eps=wl.rms_eps, max_pos=max_pos, device=dev)
    if TRACK_PARALLEL["on"]:
        import torch.distributed as dist
        m.init_random(seed=wl.seed + 100 * TRACK_PARALLEL["rank"])          # every rank its own tracks' weights
        m.set_track_group(TRACK_PARALLEL["tracks"],
                          (lambda t: dist.all_reduce(t)) if TRACK_PARALLEL["world"] > 1 else (lambda t: None))
    else:
        m.init_random(seed=wl.seed)
    return m


def timed_steps(torch, fn, steps, warmup):
    for _ in range(warmup):
        fn()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    ev0.record()
    for _ in range(steps):
        fn()
    ev1.record()
    torch.cuda.synchronize()
    return ev0.elapsed_time(ev1) / steps


def run_decode(wl, dev, steps, warmup, barrier, rank):
    import torch
    from paper_2602_07306_b200 import pt
    pk, pk_kind = peaks()
    lens_all = I.kv_lengths(wl)
    ps = wl.page_size
    model = make_model(wl, dev, max_pos=int(lens_all.max()) + 16)
    # choose the batch: everything, or the largest prefix (multiple of 16) whose pages fit
    free, _ = torch.cuda.mem_get_info(dev)
    page_bytes = wl.T * wl.L * 2 * wl.kv_heads * ps * ((wl.head_dim + 4) if kv8(wl) else wl.head_dim * 2)
    pages_of = (lens_all.astype(np.int64) + 1 + ps - 1) // ps
    budget = free - (6 << 30)
    B = wl.batch
    while B > 16 and int(pages_of[:B].sum()) * page_bytes > budget:
        B -= 16
    lens = lens_all[:B]
    num_pages = int(pages_of[:B].sum())
    cache = model.new_cache(num_pages, ps, kv_dtype="e4m3" if kv8(wl) else "model")
    seq_ids = list(range(B))
    # fill the cache by real prefills of N(0,1) inputs, grouped by length, in bounded sub-batches
    g = torch.Generator(device=dev).manual_seed(rank_batch_seed(wl.seed, rank))
    t_fill = time.time()
    order = np.argsort(-lens, kind="stable")
    i = 0
    while i < B:
        n = int(lens[order[i]])
        j = i
        while j < B and int(lens[order[j]]) == n and (j == i or (j - i + 1) * n <= 16384):
            j += 1
        ids = [int(s) for s in order[i:j]]
        x = torch.randn((wl.T, len(ids), n, wl.hidden), generator=g, device=dev, dtype=torch.float32).to(model.tdtype)
        model.prefill(cache, x, ids)
        i = j
    torch.cuda.synchronize()
    t_fill = time.time() - t_fill
    code = model.device_status()
    assert code == (0, 0), f"device status after cache fill: {code}"
    xd = torch.randn((wl.T, B, wl.hidden), generator=g, device=dev, dtype=torch.float32).to(model.tdtype)
    out = torch.empty((B, wl.hidden), dtype=torch.float32, device=dev)

    def step():
        model.decode_step(cache, xd, seq_ids, out)
        for s in seq_ids:                     # same KV lengths every step
            cache.truncate(s, int(lens[s]))

    alg = algorithmic(wl, B, lens=lens)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    barrier()
    # timed region: `value` comes from K steps with no event brackets inside; the dominant kernel's launch
    # time from K more steps, under the same clock sampler, with only that kernel's launches bracketed
    # (a bracket costs about 2 us, so bracketing every launch of a step would cost about 0.7 ms per step)
    l0 = pt.lib().pt_launch_count()
    with ClockSampler(dev) as clk:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(steps):
            step()
        ev1.record()
        torch.cuda.synchronize()
        launches = pt.lib().pt_launch_count() - l0
        model.profile(True, only=("attention",))
        for _ in range(steps):
            step()
        torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / steps
    prof = model.profile_read()
    # per-kernel breakdown from a second pass with every launch bracketed (not part of `value`)
    n_break = max(2, steps // 4)
    model.profile(True)
    for _ in range(n_break):
        step()
    torch.cuda.synchronize()
    breakdown = model.profile_read()
    model.profile(False)
    assert model.device_status() == (0, 0)
    attn_ms, attn_n = prof["attention"]
    attn_avg_ms = attn_ms / max(attn_n, 1) if attn_n else float("nan")
    achieved = alg["attn_bytes_per_layer"] / (attn_avg_ms * 1e-3) / 1e9
    ratio, why_not = decode_attn_traffic_ratio()
    if ratio is not None and not (wl.head_dim == 128 and wl.page_size == 16 and wl.dtype == "bf16" and not kv8(wl)):
        ratio, why_not = None, "counters were taken on head_dim 128, 16-token pages, bf16 cache"
    roof = {"bound": "hbm", "kernel": "k_decode_attn_e4m3" if kv8(wl) else "k_decode_attn_tma", "achieved": achieved, "peak": pk["hbm_gbs"], "unit": "GB/s",
            "frac": achieved / pk["hbm_gbs"],
            "traffic": alg["attn_bytes_per_layer"] * ratio if ratio else None, "traffic_note": why_not,
            "peak_kind": f"of {pk_kind}", "avg_launch_ms": attn_avg_ms, "launches": attn_n,
            "step_hbm_gbs": alg["bytes"] / (ms * 1e-3) / 1e9, "step_frac": alg["bytes"] / (ms * 1e-3) / 1e9 / pk["hbm_gbs"],
            "step_frac_of_nominal_8tbs": alg["bytes"] / (ms * 1e-3) / 8e12}
    # end to end from pinned host buffers
    xh = xd.cpu().pin_memory()
    oh = torch.empty((B, wl.hidden), dtype=torch.float32).pin_memory()
    xdev = torch.empty_like(xd)

    def e2e_step():
        xdev.copy_(xh, non_blocking=True)
        model.decode_step(cache, xdev, seq_ids, out)
        oh.copy_(out, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        for s in seq_ids:
            cache.truncate(s, int(lens[s]))

    for _ in range(2):
        e2e_step()
    t0 = time.perf_counter()
    n_e2e = max(3, steps // 2)
    for _ in range(n_e2e):
        e2e_step()
    e2e_ms = (time.perf_counter() - t0) / n_e2e * 1e3
    res = {"ms": ms, "tokens": B, "alg": alg, "roofline": roof, "launches": launches, "clocks": clk.summary(),
           "kernels_ms_per_step": {k: round(v[0] / n_break, 4) for k, v in breakdown.items()},
           "e2e": {"value": B / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": xh.numel() * 2,
                   "d2h_bytes_per_step": oh.numel() * 4},
           "config": {"workload": f"{wl.name}: decode T={wl.T} L={wl.L} D={wl.D} H={wl.hidden} heads={wl.heads}/{wl.kv_heads} "
                                  f"F={wl.ffn} batch={B} kv_len={'U[%d,%d]' % wl.ragged if wl.ragged else wl.seq} page={ps}"
                                  f" cache={'e4m3 codes + fp32 scale per vector' if kv8(wl) else 'bf16'}",
                      "batch": B, "batch_requested": wl.batch, "kv_tokens": int(lens.sum()), "cache_fill_s": round(t_fill, 2),
                      "l2": "working set (KV cache + weights) far larger than L2; no flush needed"}}
    cache.close()
    model.close()
    del cache, model
    torch.cuda.empty_cache()
    return res


def run_prefill(wl, dev, steps, warmup, barrier, rank):
    import torch
    from paper_2602_07306_b200 import pt
    pk, pk_kind = peaks()
    B, S, ps = wl.batch, wl.seq, wl.page_size
    model = make_model(wl, dev, max_pos=S)
    pages = B * ((S + ps - 1) // ps)
    cache = model.new_cache(pages, ps)
    seq_ids = list(range(B))
    g = torch.Generator(device=dev).manual_seed(rank_batch_seed(wl.seed, rank))
    x = torch.randn((wl.T, B, S, wl.hidden), generator=g, device=dev, dtype=torch.float32).to(model.tdtype)
    out = torch.empty((B, S, wl.hidden), dtype=torch.float32, device=dev)

    def step():
        model.prefill(cache, x, seq_ids, out)
        for s in seq_ids:
            cache.truncate(s, 0)

    alg = algorithmic(wl, B, S=S)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    barrier()
    # `value` from K steps with no event brackets inside; the per-kernel times from K more steps, under the
    # same clock sampler, with every launch bracketed
    l0 = pt.lib().pt_launch_count()
    with ClockSampler(dev) as clk:
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record()
        for _ in range(steps):
            step()
        ev1.record()
        torch.cuda.synchronize()
        launches = pt.lib().pt_launch_count() - l0
        model.profile(True)
        for _ in range(steps):
            step()
        torch.cuda.synchronize()
    ms = ev0.elapsed_time(ev1) / steps
    prof = model.profile_read()
    model.profile(False)
    assert model.device_status() == (0, 0)
    gemm_ms = sum(prof[k][0] for k in ("gemm_qkv", "gemm_out", "gemm_gate_up", "gemm_down", "gemm_down_sync")) / steps
    gemm_n = sum(prof[k][1] for k in ("gemm_qkv", "gemm_out", "gemm_gate_up", "gemm_down", "gemm_down_sync"))
    attn_ms = prof["attention"][0] / steps
    if gemm_n == 0:        # the fp32 workload runs the plain kernels, which are not bracketed per category
        gemm_ms, attn_ms = float("nan"), float("nan")
    gemm_tf = alg["gemm_flops"] / (gemm_ms * 1e-3) / 1e12
    attn_tf = alg["attn_flops"] / (attn_ms * 1e-3) / 1e12
    peak = pk["bf16_tflops_sustained"] if ms * steps > 1000 else pk["bf16_tflops"]
    if gemm_n == 0:
        step_tf = alg["flops"] / (ms * 1e-3) / 1e12
        roof = {"bound": "alu", "kernel": "plain fp32 kernels (launch-bound workload: absolute numbers only)", "achieved": step_tf,
                "peak": None, "unit": "TFLOP/s", "frac": None, "traffic": None, "peak_kind": "not applicable"}
    else:
      roof = {"bound": "tensor", "kernel": "gemm_tc (QKV, out, gate/up, down, down+sync)", "achieved": gemm_tf, "peak": peak,
            "unit": "TFLOP/s", "frac": gemm_tf / peak, "traffic": None, "peak_kind": f"of {pk_kind}",
            "avg_launch_ms": gemm_ms * steps / max(gemm_n, 1), "launches": gemm_n,
            "frac_of_nominal_2250": gemm_tf / 2250.0, "attention_tflops": attn_tf,
            "step_tflops": alg["flops"] / (ms * 1e-3) / 1e12}
    xh = x.cpu().pin_memory()
    oh = torch.empty((B, S, wl.hidden), dtype=torch.float32).pin_memory()
    xdev = torch.empty_like(x)

    def e2e_step():
        xdev.copy_(xh, non_blocking=True)
        model.prefill(cache, xdev, seq_ids, out)
        oh.copy_(out, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        for s in seq_ids:
            cache.truncate(s, 0)

    e2e_step()
    t0 = time.perf_counter()
    n_e2e = max(2, steps // 2)
    for _ in range(n_e2e):
        e2e_step()
    e2e_ms = (time.perf_counter() - t0) / n_e2e * 1e3
    res = {"ms": ms, "tokens": B * S, "alg": alg, "roofline": roof, "launches": launches, "clocks": clk.summary(),
           "kernels_ms_per_step": {k: round(v[0] / steps, 4) for k, v in prof.items()},
           "e2e": {"value": B * S / (e2e_ms * 1e-3), "unit": "tokens/s", "h2d_bytes_per_step": xh.numel() * 2,
                   "d2h_bytes_per_step": oh.numel() * 4},
           "config": {"workload": f"{wl.name}: prefill T={wl.T} L={wl.L} D={wl.D} H={wl.hidden} heads={wl.heads}/{wl.kv_heads} "
                                  f"F={wl.ffn} batch={B} seq={S} page={ps}", "batch": B, "seq_len": S,
                      "l2": "activations + weights per step larger than L2" if wl.T * B * S * wl.hidden * 4 > 126e6
                            else "inputs smaller than L2: weights partly L2-resident between steps (launch-bound workload)"}}
    cache.close()
    model.close()
    del cache, model
    torch.cuda.empty_cache()
    return res


# ------------------------------------------------------------------------------ CPU oracle arm

class _Cached:
    def __init__(self, src, T, L):
        self.w = {(t, l): src.get(t, l) for l in range(L) for t in range(T)}

    def get(self, t, l):
        return self.w[(t, l)]


_SAMPLE_WEIGHTS = {}          # the sample's weights are drawn once per process, outside every timed call


def oracle_sample(wl, budget_s=20.0):
    """Time the CPU oracle, as it stands, on a bounded sample of the workload: the first track
    block (D of the L layers, all T tracks) on a few rows / a shorter prompt; tokens/s is scaled by
    D/L to the full depth (layers cost the same).  Returns (tokens_per_s, description, seconds)."""
    from oracle import pt_oracle as O
    import dataclasses
    cores = len(os.sched_getaffinity(0))
    sub = dataclasses.replace(wl, L=wl.D)
    cfg = O.PTConfig(T=sub.T, D=sub.D, L=sub.L, hidden=sub.hidden, heads=sub.heads, kv_heads=sub.kv_heads, ffn=sub.ffn)
    key = (sub.name, sub.T, sub.L, sub.hidden, sub.ffn, sub.seed)
    if key not in _SAMPLE_WEIGHTS:
        _SAMPLE_WEIGHTS[key] = _Cached(I.WeightSource(sub), sub.T, sub.L)
    ws = _SAMPLE_WEIGHTS[key]
    scale = wl.D / wl.L
    if wl.mode == "decode":
        rows = 2
        lens = I.kv_lengths(wl, batch=rows)
        pages = int(sum((int(n) + 1 + 15) // 16 for n in lens))
        ckey = key + ("cache",)
        if ckey not in _SAMPLE_WEIGHTS:               # the pre-filled cache too is built once, outside the timed calls
            cache = O.PagedKVCache(cfg, pages, 16)
            rng = np.random.default_rng(0)
            for b in range(rows):                     # synthetic cache contents: timing does not depend on them
                cache.reserve(b, int(lens[b]) + 1)
            cache.pool[...] = rng.standard_normal(cache.pool.shape)
            _SAMPLE_WEIGHTS[ckey] = cache
        cache = _SAMPLE_WEIGHTS[ckey]
        for b in range(rows):
            cache.length[b] = int(lens[b])            # every timed step decodes at the same KV lengths
        x = I.decode_inputs(sub, batch=rows)
        t0 = time.perf_counter()
        O.pt_decode_step(cfg, ws, x, cache, list(range(rows)))
        dt = time.perf_counter() - t0
        return rows / dt * scale, (f"{rows} sequences (KV {lens.tolist()}), first track block ({wl.D} of {wl.L} layers, "
                                   f"all {wl.T} tracks), cache pre-filled with N(0,1); tokens/s scaled by {wl.D}/{wl.L}"), dt, cores
    S = min(wl.seq, 256)
    x = I.prefill_inputs(sub, batch=1, seq=S)
    cache = O.PagedKVCache(cfg, (S + 15) // 16, 16)
    t0 = time.perf_counter()
    O.pt_prefill(cfg, ws, x, cache, [0])
    dt = time.perf_counter() - t0
    return S / dt * scale, (f"1 sequence x {S} tokens, first track block ({wl.D} of {wl.L} layers, all {wl.T} tracks); "
                            f"tokens/s scaled by {wl.D}/{wl.L}"), dt, cores


# ------------------------------------------------------------------------------ ranks

def rank_batch_seed(seed, rank):
    """Seed of the inputs of one rank's batch: rank r owns sequences [r*B, (r+1)*B) of the job's
    global batch, drawn from its own stream; the model weights are the same on every rank."""
    return int(seed) + 1 + 7919 * int(rank)


def aggregate_over_ranks(ms, tokens, e2e_tokens_per_s, world, device):
    """Whole-job numbers of a weak-scaling run: every rank processed `tokens` tokens per step on
    its own batch in `ms` device milliseconds (no data-path collective).  The job's step time is
    the slowest rank's, the job's tokens are the sum; the same for the end-to-end leg.  Only
    these three scalars cross ranks.  Returns (ms, total_tokens, e2e_tokens_per_s)."""
    if world <= 1:
        return float(ms), float(tokens), float(e2e_tokens_per_s)
    import torch
    import torch.distributed as dist
    tmax = torch.tensor([float(ms), float(tokens) / float(e2e_tokens_per_s)], dtype=torch.float64, device=device)
    dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
    toks = torch.tensor([float(tokens)], dtype=torch.float64, device=device)
    dist.all_reduce(toks, op=dist.ReduceOp.SUM)
    total = float(toks.item())
    return float(tmax[0].item()), total, total / float(tmax[1].item())


def aggregate_track_ranks(ms, tokens, e2e_tokens_per_s, world, device):
    """Whole-job numbers of a track-parallel run: every rank holds T / world tracks of ONE model and
    all ranks process the same batch, so the job's tokens are one rank's (not the sum) and its step
    time is the slowest rank's; the same for the end-to-end leg.  Returns (ms, tokens, e2e_tokens_per_s)."""
    ms_max, total, e2e_sum_over_max = aggregate_over_ranks(ms, tokens, e2e_tokens_per_s, world, device)
    return ms_max, total / world, e2e_sum_over_max / world


# ------------------------------------------------------------------------------ main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2")
    ap.add_argument("--extra", default="cfg3,cfg4,cfg4_kv8,cfg2_kv8,cfg1,cfg0", help="comma-separated workloads reported under 'extra' (N=1 only); '' for none")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--parallel", default="replicas", choices=["replicas", "tracks"],
                    help="N > 1: 'replicas' = every rank runs the whole model on its own batch (weak scaling, no collective); "
                         "'tracks' = every rank holds T/N tracks of one model and all ranks share the batch (strong scaling, "
                         "one all-reduce per track block)")
    ap.add_argument("--seq", type=int, default=0, help="override the workload's sequence / KV length")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch")
    ap.add_argument("--depth", type=int, default=0, help="override the track-block depth D (must divide L)")
    a = ap.parse_args()
    a.warmup = max(a.warmup, 3) if a.impl == "ours" else a.warmup
    wl = I.WORKLOADS[a.workload]
    import dataclasses
    over = {k: v for k, v in (("seq", a.seq), ("batch", a.batch), ("D", a.depth)) if v}
    if over:
        wl = dataclasses.replace(wl, **over)
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    metric = "decode tokens/s" if wl.mode == "decode" else "prefill tokens/s"

    if a.impl == "reference":
        if rank != 0:
            return
        vals = []
        for _ in range(max(1, a.warmup)):
            oracle_sample(wl)
        t0 = time.perf_counter()
        for _ in range(a.steps):
            v, sample, dt, cores = oracle_sample(wl)
            vals.append(v)
        ms = (time.perf_counter() - t0) / a.steps * 1e3
        v = float(np.mean(vals))
        print(json.dumps({"impl": "reference", "metric": f"PT {metric}", "value": v, "unit": "tokens/s",
                          "n_gpus": a.gpus, "steps": a.steps, "warmup": a.warmup, "ms_per_step": ms, "higher_is_better": True,
                          "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
                          "config": {"workload": f"{wl.name} ({wl.mode})"},
                          "cpu_baseline": {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample},
                          "e2e": {"value": v, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}))
        return

    import torch
    import torch.distributed as dist
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    run = run_decode if wl.mode == "decode" else run_prefill
    tracks_mode = a.parallel == "tracks"
    if tracks_mode:
        # one model over all ranks: each holds T / N tracks, all see the same batch (same input seed),
        # so the job's tokens are one rank's and the step time is the slowest rank's
        assert wl.T % world == 0, "the number of ranks must divide the number of tracks"
        TRACK_PARALLEL.update(on=True, world=world, rank=rank, tracks=wl.T)
        r = run(dataclasses.replace(wl, T=wl.T // world), dev, a.steps, a.warmup, barrier, 0)
        ms, total_tokens, e2e_value = aggregate_track_ranks(r["ms"], r["tokens"], r["e2e"]["value"], world, dev)
        r["config"]["parallelism"] = f"tracks: {wl.T} tracks over {world} rank(s), one all-reduce per track block"
    else:
        r = run(wl, dev, a.steps, a.warmup, barrier, rank)
        ms, total_tokens, e2e_value = aggregate_over_ranks(r["ms"], r["tokens"], r["e2e"]["value"], world, dev)
    r["e2e"]["value"] = e2e_value
    extra = {}
    if world == 1 and a.extra and not tracks_mode:
        for name in [n for n in a.extra.split(",") if n and n != a.workload]:
            w2 = I.WORKLOADS[name]
            try:
                r2 = (run_decode if w2.mode == "decode" else run_prefill)(w2, dev, max(10, a.steps // 2), 3, barrier, rank)
                extra[name] = {"metric": "decode tokens/s" if w2.mode == "decode" else "prefill tokens/s",
                               "value": r2["tokens"] / (r2["ms"] * 1e-3), "ms_per_step": r2["ms"], "roofline": r2["roofline"],
                               "kernels_ms_per_step": r2["kernels_ms_per_step"], "config": r2["config"], "clocks": r2["clocks"],
                               "e2e": r2["e2e"]}
            except Exception as e:  # an extra must never take the headline down
                extra[name] = {"error": repr(e)[:300]}
    cpu = None
    if rank == 0 and world == 1 and not a.no_cpu_baseline:
        v, sample, dt, cores = oracle_sample(wl)
        cpu = {"value": v, "unit": "tokens/s", "cores": cores, "kind": "oracle", "sample": sample, "seconds": round(dt, 2)}
    if rank == 0:
        line = {"metric": f"PT {metric}", "value": total_tokens / (ms * 1e-3), "unit": "tokens/s", "n_gpus": world,
                "steps": a.steps, "warmup": a.warmup, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "strong" if tracks_mode else "weak",
                "vs_baseline": None, "dtype": "bf16" if wl.dtype == "bf16" else "f32", "data": "synthetic",
                "config": r["config"], "clocks": r["clocks"], "e2e": r["e2e"], "gpu_launches": int(r["launches"]),
                "roofline": r["roofline"], "cpu_baseline": cpu, "kernels_ms_per_step": r["kernels_ms_per_step"],
                "algorithmic": r["alg"], "extra": extra}
        print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
