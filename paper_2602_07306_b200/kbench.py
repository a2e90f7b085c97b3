"""Time one kernel of the PT forward pass through its kernel-level C-ABI entry point.

    python -m paper_2602_07306_b200.kbench decode --T 8 --B 64 --nq 8 --nkv 8 --dh 128 --len 2048
    python -m paper_2602_07306_b200.kbench prefill --T 8 --B 8 --S 4096 --nq 8 --nkv 8 --dh 128 [--impl 1]
    python -m paper_2602_07306_b200.kbench layer --T 8 --B 2 --S 4096 --H 1024 --nq 8 --nkv 8 --F 2816
    python -m paper_2602_07306_b200.kbench generate --B 1 --S 1024 --new 64 [--depth 2|4|8]
    python -m paper_2602_07306_b200.kbench gemm --T 8 --M 32768 --N 3072 --K 1024 [--bn 256] [--fold]
    python -m paper_2602_07306_b200.kbench step --T 4 --B 64 --len 2048 --H 2048 --nq 16 --nkv 4 --F 5632 [--kv8 1 [--mma_sync 1]]

Prints one JSON line: average device time per launch (CUDA events on the launching stream,
after warm-up) and the achieved GB/s (decode: K/V bytes read) or TFLOP/s (gemm).  Small cases of
the same commands are what the ncu summaries under profiles/ were captured on.
"""
from __future__ import annotations

import argparse
import json

import numpy as np
import torch

from paper_2602_07306_b200 import pt


def decode(a):
    dev = torch.device("cuda:0")
    ps = a.ps
    lens = [a.len] * a.B if a.ragged == 0 else np.random.default_rng(0).integers(a.ragged, a.len + 1, a.B).tolist()
    maxp = max(-(-n // ps) for n in lens)
    pages = sum(-(-n // ps) for n in lens)
    g = torch.Generator(device=dev).manual_seed(0)
    pool = torch.randn((a.T, pages, 2, a.nkv, ps, a.dh), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    q = torch.randn((a.T, a.B, a.nq * a.dh), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    perm = torch.randperm(pages, generator=torch.Generator().manual_seed(0)).to(torch.int32)
    bt = torch.zeros((a.B, maxp), dtype=torch.int32)
    nxt = 0
    for b, n in enumerate(lens):
        k = -(-n // ps)
        bt[b, :k] = perm[nxt:nxt + k]
        nxt += k
    bt = bt.to(dev)
    n = pt._SZ()
    pt.check(pt.lib().pt_kernel_decode_attn_scratch_bytes(a.T, a.B, a.nq, a.dh, pt.C.byref(n)))
    scratch = torch.empty(n.value, dtype=torch.uint8, device=dev)
    for _ in range(a.warmup):
        out, status = pt.kernel_decode_attn(q, pool, bt, lens, nq=a.nq, nkv=a.nkv, dh=a.dh, ps=ps, scratch=scratch)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        out, status = pt.kernel_decode_attn(q, pool, bt, lens, nq=a.nq, nkv=a.nkv, dh=a.dh, ps=ps, scratch=scratch)
    e1.record()
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0]
    ms = e0.elapsed_time(e1) / a.iters
    byts = a.T * 2 * a.nkv * a.dh * 2 * sum(lens)
    print(json.dumps({"kernel": "decode_attn", "ms": ms, "GBps": byts / ms / 1e6, "bytes": byts, "args": vars(a)}))


def prefill(a):
    dev = torch.device("cuda:0")
    ps = a.ps
    n = a.S + a.start
    maxp = -(-n // ps)
    pages = a.B * maxp
    g = torch.Generator(device=dev).manual_seed(0)
    pool = torch.randn((a.T, pages, 2, a.nkv, ps, a.dh), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    q = torch.randn((a.T, a.B * a.S, a.nq * a.dh), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    perm = torch.randperm(pages, generator=torch.Generator().manual_seed(0)).to(torch.int32)
    bt = perm.reshape(a.B, maxp).contiguous().to(dev)
    lens = torch.full((a.B,), n, dtype=torch.int32, device=dev)
    run = lambda: pt.kernel_prefill_attn(q, pool, bt, lens, S=a.S, nq=a.nq, nkv=a.nkv, dh=a.dh, ps=ps, impl=a.impl)
    for _ in range(a.warmup):
        out, status = run()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        out, status = run()
    e1.record()
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0], status[:2].tolist()
    ms = e0.elapsed_time(e1) / a.iters
    # causal triangle only: row s sees start + s + 1 keys
    keys = a.S * a.start + a.S * (a.S + 1) // 2
    flops = 4.0 * a.T * a.B * a.nq * a.dh * keys
    print(json.dumps({"kernel": "prefill_attn", "ms": ms, "TFLOPs": flops / ms / 1e9, "args": vars(a)}))


def layer(a):
    """One PT layer of the given width (all tracks, L = D = 1) as a prefill: the four fused GEMMs and the
    attention kernel in their real launch configuration, small enough to capture under a profiler.  With
    --layers 2 the track block is two layers deep, so the first layer's down GEMM is the plain one (gemm_down)."""
    from paper_2602_07306_b200 import inputs as I
    dev = torch.device("cuda:0")
    m = pt.Model(T=a.T, D=a.layers, L=a.layers, hidden=a.H, heads=a.nq, kv_heads=a.nkv, ffn=a.F, dtype="bf16", max_pos=a.S,
                 experts=a.experts, top_k=a.top_k, device=dev)
    m.init_random(0)
    cache = m.new_cache(a.B * (-(-a.S // a.ps)), a.ps)
    g = torch.Generator(device=dev).manual_seed(0)
    x = torch.randn((a.T, a.B, a.S, a.H), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty((a.B, a.S, a.H), dtype=torch.float32, device=dev)
    ids = list(range(a.B))

    def step():
        m.prefill(cache, x, ids, out)
        for s_ in ids:
            cache.truncate(s_, 0)
    for _ in range(a.warmup):
        step()
    torch.cuda.synchronize()
    m.profile(True)
    for _ in range(a.iters):
        step()
    torch.cuda.synchronize()
    prof = m.profile_read()
    assert m.device_status() == (0, 0)
    tok = a.B * a.S
    kx = max(a.top_k, 1)          # PT-MoE: a token's feed-forward flops are those of its top_k experts
    fl = {"gemm_qkv": 2.0 * a.T * tok * a.H * (a.nq + 2 * a.nkv) * (a.H // a.nq), "gemm_out": 2.0 * a.T * tok * a.H * a.H,
          "gemm_gate_up": 4.0 * a.T * tok * a.H * a.F * kx, "gemm_down_sync": 2.0 * a.T * tok * a.H * a.F * kx,
          "gemm_down": 2.0 * a.T * tok * a.H * a.F * kx}
    res = {k: {"ms": v[0] / max(v[1], 1), "TFLOPs": fl[k] / (v[0] / max(v[1], 1)) / 1e9 if k in fl and v[1] else None}
           for k, v in prof.items() if v[1]}
    print(json.dumps({"kernel": "layer", "per_launch": res, "args": vars(a)}))


def step(a):
    """Decode steps of a small model (L = D = --layers) of the given width over a cache filled by real prefills, with
    the cache in the model dtype or (--kv8 1) in the E4M3 format: per-category device time per launch, and the
    achieved rate of the attention kernel over the bytes of the cached vectors it reads."""
    dev = torch.device("cuda:0")
    m = pt.Model(T=a.T, D=a.layers, L=a.layers, hidden=a.H, heads=a.nq, kv_heads=a.nkv, ffn=a.F, dtype="bf16",
                 max_pos=a.len + 16, flags=4 if a.mma_sync else 0, device=dev)
    m.init_random(0)
    dh = a.H // a.nq
    cache = m.new_cache(a.B * (-(-(a.len + 1) // a.ps)), a.ps, kv_dtype="e4m3" if a.kv8 else "model")
    g = torch.Generator(device=dev).manual_seed(0)
    sub = max(1, 8192 // a.len)
    for i in range(0, a.B, sub):
        ids = list(range(i, min(a.B, i + sub)))
        x = torch.randn((a.T, len(ids), a.len, a.H), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
        m.prefill(cache, x, ids)
    xd = torch.randn((a.T, a.B, a.H), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    out = torch.empty((a.B, a.H), dtype=torch.float32, device=dev)
    ids = list(range(a.B))

    def one():
        m.decode_step(cache, xd, ids, out)
        for s_ in ids:
            cache.truncate(s_, a.len)
    for _ in range(a.warmup):
        one()
    torch.cuda.synchronize()
    m.profile(True)
    for _ in range(a.iters):
        one()
    torch.cuda.synchronize()
    prof = m.profile_read()
    assert m.device_status() == (0, 0)
    vec = dh + 4 if a.kv8 else 2 * dh
    byts = a.T * 2 * a.nkv * vec * a.B * (a.len + 1)
    res = {k: v[0] / max(v[1], 1) for k, v in prof.items() if v[1]}
    print(json.dumps({"kernel": "decode_step", "ms_per_launch": res, "attention_GBps": byts / res["attention"] / 1e6,
                      "attention_bytes": byts, "args": vars(a)}))


def generate(a):
    """Greedy generation at the head layout of the paper's 30B model (inputs.WORKLOADS["pt30b_prefill"]): time
    to the first token (embed + prefill + LM head + choice) and time per further token, batch a.B."""
    from paper_2602_07306_b200 import inputs as I
    import dataclasses
    wl = I.WORKLOADS["pt30b_prefill"]
    if a.depth:
        wl = dataclasses.replace(wl, D=a.depth)
    dev = torch.device("cuda:0")
    m = pt.Model(T=wl.T, D=wl.D, L=wl.L, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads, ffn=wl.ffn,
                 dtype="bf16", max_pos=a.S + a.new + 16, device=dev)
    m.init_random(0)
    g = torch.Generator(device=dev).manual_seed(0)
    H = wl.hidden
    m.load_lm(torch.randn((a.vocab, H), generator=g, device=dev), torch.randn((a.vocab, H), generator=g, device=dev) * 0.05,
              torch.ones(H, device=dev))
    pages = a.B * (-(-(a.S + a.new) // 16))
    cache = m.new_cache(pages, 16)
    prompt = torch.randint(0, a.vocab, (a.B, a.S), generator=g, device=dev, dtype=torch.int32)
    ids = list(range(a.B))

    def run(n_new):
        for s_ in ids:
            if cache.length(s_):
                cache.truncate(s_, 0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        toks, _ = m.generate(cache, prompt, n_new, ids)
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)
    for _ in range(a.warmup):
        run(2)
    ttft = min(run(1) for _ in range(a.iters))
    full = min(run(1 + a.new) for _ in range(a.iters))
    assert m.device_status() == (0, 0)
    print(json.dumps({"kernel": "generate", "ttft_ms": ttft, "tpot_ms": (full - ttft) / a.new, "tokens_per_s": a.B * a.new / ((full - ttft) * 1e-3),
                      "model": f"T={wl.T} L={wl.L} D={wl.D} H={wl.hidden} heads={wl.heads}/{wl.kv_heads} F={wl.ffn} vocab={a.vocab}", "args": vars(a)}))


def gemm(a):
    """The GEMM alone (plain epilogue).  Output and status are allocated once, so the loop is launches only; with few
    rows the interesting figure is W_GBps, the rate at which the weights stream from HBM (choose N so that W exceeds L2)."""
    dev = torch.device("cuda:0")
    g = torch.Generator(device=dev).manual_seed(0)
    A = torch.randn((a.T, a.M, a.K), generator=g, device=dev, dtype=torch.float32).to(torch.bfloat16)
    W = (torch.randn((a.T, a.N, a.K), generator=g, device=dev, dtype=torch.float32) * 0.05).to(torch.bfloat16)
    c = torch.empty((1 if a.fold else a.T, a.M, a.N), dtype=torch.float32, device=dev)
    status = torch.zeros(16, dtype=torch.int32, device=dev)
    stream = torch.cuda.current_stream().cuda_stream

    def launch():
        pt.check(pt.lib().pt_kernel_gemm_bf16(A.data_ptr(), W.data_ptr(), c.data_ptr(), a.T, a.M, a.N, a.K, a.bn, int(a.fold),
                                               status.data_ptr(), stream))
    for _ in range(a.warmup):
        launch()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(a.iters):
        launch()
    e1.record()
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0]
    ms = e0.elapsed_time(e1) / a.iters
    flops = 2.0 * a.T * a.M * a.N * a.K
    print(json.dumps({"kernel": "gemm_bf16", "ms": ms, "TFLOPs": flops / ms / 1e9, "W_GBps": W.numel() * 2 / ms / 1e6, "args": vars(a)}))


def main():
    ap = argparse.ArgumentParser()
    sub = ap.add_subparsers(dest="cmd", required=True)
    d = sub.add_parser("decode")
    for k, v in dict(T=8, B=64, nq=8, nkv=8, dh=128, len=2048, ps=16, ragged=0, iters=20, warmup=3).items():
        d.add_argument("--" + k, type=int, default=v)
    pf = sub.add_parser("prefill")
    for k, v in dict(T=8, B=8, S=4096, start=0, nq=8, nkv=8, dh=128, ps=16, impl=0, iters=10, warmup=3).items():
        pf.add_argument("--" + k, type=int, default=v)
    ly = sub.add_parser("layer")
    for k, v in dict(T=8, B=2, S=4096, H=1024, nq=8, nkv=8, F=2816, ps=16, layers=1, experts=0, top_k=0, iters=3, warmup=1).items():
        ly.add_argument("--" + k, type=int, default=v)
    gn = sub.add_parser("generate")
    for k, v in dict(B=1, S=1024, new=64, vocab=32000, depth=0, iters=3, warmup=1).items():
        gn.add_argument("--" + k, type=int, default=v)
    sp = sub.add_parser("step")
    for k, v in dict(T=4, B=64, len=2048, H=2048, nq=16, nkv=4, F=5632, ps=16, layers=2, kv8=0, mma_sync=0, iters=10, warmup=3).items():
        sp.add_argument("--" + k, type=int, default=v)
    gm = sub.add_parser("gemm")
    for k, v in dict(T=8, M=4096, N=3072, K=1024, bn=0, iters=20, warmup=3).items():
        gm.add_argument("--" + k, type=int, default=v)
    gm.add_argument("--fold", action="store_true")
    a = ap.parse_args()
    {"decode": decode, "gemm": gemm, "prefill": prefill, "layer": layer, "generate": generate, "step": step}[a.cmd](a)


if __name__ == "__main__":
    main()
