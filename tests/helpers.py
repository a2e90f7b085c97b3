"""Shared test plumbing: run the same seeded workload through the CPU oracle and the C ABI."""
import numpy as np

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I


def oracle_cfg(wl, sync_op="sum"):
    return O.PTConfig(T=wl.T, D=wl.D, L=wl.L, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads,
                      ffn=wl.ffn, rope_base=wl.rope_base, rms_eps=wl.rms_eps, sync_op=sync_op)


def make_model(wl, ws, sync_op="sum", max_pos=4096, simt=False):
    from paper_2602_07306_b200 import pt
    m = pt.Model(T=wl.T, D=wl.D, L=wl.L, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads, ffn=wl.ffn,
                 dtype=wl.dtype, rope_base=wl.rope_base, rms_eps=wl.rms_eps, sync_op=sync_op,
                 max_pos=max_pos, simt=simt)
    m.load(ws)
    return m


def to_dev(model, a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).to(model.device).to(model.tdtype).contiguous()


def rel_errs(got, ref):
    got = np.asarray(got, np.float64)
    ref = np.asarray(ref, np.float64)
    d = np.abs(got - ref)
    return d.max() / max(np.abs(ref).max(), 1e-300), d.mean() / max(np.abs(ref).mean(), 1e-300)


def tol(dtype):
    """(max-abs / max|ref|, mean-abs / mean|ref|) bounds: fp32 path 1e-4; bf16 path 2e-2 and 2e-3."""
    return (1e-4, 1e-4) if dtype == "f32" else (2e-2, 2e-3)


# Mean-error bounds for the wide models.  With per-track hidden 1024 or 2048 the layer deltas are as
# large as the stream itself, and rounding only what must be bf16 (the GEMM and attention operands and
# the cache) in otherwise exact arithmetic already gives a mean relative error above the 2e-3 target
# once a track block has run: tests/test_bf16_floor.py measures that floor on the CPU.  At those
# widths the CUDA path is held to the floor plus a margin instead.
DEEP_MEAN_TOL = 3.0e-3        # hidden 1024 (the T=8, L=32 model)
WIDE_MEAN_TOL = 3.5e-3        # hidden 2048 (the T=4, L=48 GQA model)


def assert_close(got, ref, dtype, what="", mean_tol=None):
    mx, mean = rel_errs(got, ref)
    tmx, tmean = tol(dtype)
    if mean_tol is not None:
        tmean = mean_tol
    assert np.all(np.isfinite(np.asarray(got, np.float64))), f"{what}: non-finite values"
    assert mx <= tmx and mean <= tmean, f"{what}: max-rel {mx:.3e} (<= {tmx}), mean-rel {mean:.3e} (<= {tmean})"
    return mx, mean


def pool_as_numpy(cache, wl):
    """Device pool -> float64 array [T, L, pages, 2, nkv, page, dh]."""
    import torch
    p = cache.pool.to(torch.float32).cpu().numpy().astype(np.float64)
    return p.reshape(wl.T, wl.L, cache.num_pages, 2, wl.kv_heads, cache.page_size, wl.head_dim)
