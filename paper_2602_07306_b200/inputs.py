"""Seeded synthetic inputs for the Parallel Track (PT) forward pass.

This module only draws numbers and describes workloads; it holds none of the
method's arithmetic, so both the CPU oracle's tests and the CUDA path's tests
may use it.  Every tensor has its own stream: NumPy ``Generator(PCG64)`` seeded
with ``SeedSequence([seed, kind, track, layer])`` and drawn in float32, so any
(track, layer) can be regenerated on demand without holding a whole model.

Recipe (the five workloads): weights N(0, 0.02), norm gains 1, hidden-state
inputs N(0, 1).  For the bf16 workloads the float32 draws are rounded to
bfloat16 (round-to-nearest-even) once, here, and every consumer sees the
rounded values.
"""
from __future__ import annotations

from dataclasses import dataclass, field
import numpy as np

# tensor kinds, also the draw order inside one (track, layer)
KINDS = ("wq", "wk", "wv", "wo", "wg", "wu", "wd", "g1", "g2", "wr")     # wr: the router of a PT-MoE layer (only with experts > 0)
_KIND_ID = {k: i for i, k in enumerate(KINDS)}
_KIND_X = 100        # prefill inputs
_KIND_XDEC = 101     # decode inputs
_KIND_LENS = 102     # ragged KV lengths
_KIND_PERM = 103     # free-list permutation


def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """float32 -> nearest bfloat16 (ties to even), returned as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    bias = ((u >> 16) & 1) + np.uint32(0x7FFF)
    r = ((u + bias) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """float32 values that are exactly representable in bf16 -> uint16 bit patterns."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    return (a.view(np.uint32) >> 16).astype(np.uint16)


def bits_to_f32(b: np.ndarray) -> np.ndarray:
    """uint16 bf16 bit patterns -> float32."""
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << 16).view(np.float32)


def _rng(seed: int, kind: int, a: int = 0, b: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, kind, a, b])))


@dataclass(frozen=True)
class Workload:
    """One workload: architecture numbers plus batch geometry."""
    name: str
    T: int
    L: int
    D: int
    hidden: int
    heads: int
    kv_heads: int
    ffn: int
    dtype: str            # "f32" or "bf16"
    mode: str             # "prefill" or "decode"
    batch: int
    seq: int              # prefill: tokens per sequence; decode: KV length before the step (0 if ragged)
    ragged: tuple = ()    # (lo, hi) inclusive for ragged decode
    page_size: int = 16
    rope_base: float = 10000.0
    rms_eps: float = 1e-6
    seed: int = 0
    experts: int = 0      # > 0: PT-MoE - every track's feed-forward is a mixture of `experts` experts of width ffn
    top_k: int = 0

    @property
    def head_dim(self) -> int:
        return self.hidden // self.heads

    def weight_shape(self, kind: str) -> tuple:
        H, dh, F = self.hidden, self.head_dim, self.ffn
        E = (self.experts,) if self.experts else ()
        return {
            "wq": (self.heads * dh, H), "wk": (self.kv_heads * dh, H), "wv": (self.kv_heads * dh, H),
            "wo": (H, self.heads * dh), "wg": E + (F, H), "wu": E + (F, H), "wd": E + (H, F),
            "g1": (H,), "g2": (H,), "wr": (max(self.experts, 1), H),
        }[kind]

    def params_per_track_layer(self) -> int:
        H, dh, F = self.hidden, self.head_dim, self.ffn * max(self.experts, 1)
        return 2 * H * self.heads * dh + 2 * H * self.kv_heads * dh + 3 * H * F


WORKLOADS = {
    "cfg0": Workload("cfg0", T=2, L=4, D=2, hidden=128, heads=4, kv_heads=4, ffn=512,
                     dtype="f32", mode="prefill", batch=1, seq=64),
    "cfg1": Workload("cfg1", T=4, L=8, D=4, hidden=512, heads=8, kv_heads=8, ffn=1376,
                     dtype="bf16", mode="prefill", batch=4, seq=512),
    "cfg2": Workload("cfg2", T=8, L=32, D=8, hidden=1024, heads=8, kv_heads=8, ffn=2816,
                     dtype="bf16", mode="decode", batch=64, seq=2048),
    "cfg3": Workload("cfg3", T=8, L=32, D=8, hidden=1024, heads=8, kv_heads=8, ffn=2816,
                     dtype="bf16", mode="prefill", batch=8, seq=4096),
    "cfg4": Workload("cfg4", T=4, L=48, D=6, hidden=2048, heads=16, kv_heads=4, ffn=5632,
                     dtype="bf16", mode="decode", batch=256, seq=0, ragged=(512, 4096)),
    # The batched decode workload with the cache in the library's E4M3 format.
    "cfg2_kv8": Workload("cfg2_kv8", T=8, L=32, D=8, hidden=1024, heads=8, kv_heads=8, ffn=2816,
                         dtype="bf16", mode="decode", batch=64, seq=2048),
    # The same ragged decode workload with the cache in the library's E4M3 format: the whole batch of 256 fits.
    "cfg4_kv8": Workload("cfg4_kv8", T=4, L=48, D=6, hidden=2048, heads=16, kv_heads=4, ffn=5632,
                         dtype="bf16", mode="decode", batch=256, seq=0, ragged=(512, 4096)),
    # The head layout of the paper's 30B PT model (Table 1: 8 tracks, 48 layers, 8 query heads and 1 KV
    # head per track, block depth D in {2, 4, 8}) at the request shapes of its latency tables (batch 1,
    # 1024 .. 63488 prompt tokens).  The paper gives neither the hidden nor the feed-forward width: 8
    # heads of 128 fix hidden 1024 here and the feed-forward width 4096 is this repository's choice.
    "pt30b_prefill": Workload("pt30b_prefill", T=8, L=48, D=8, hidden=1024, heads=8, kv_heads=1, ffn=4096,
                              dtype="bf16", mode="prefill", batch=1, seq=16384),
    "pt30b_decode": Workload("pt30b_decode", T=8, L=48, D=8, hidden=1024, heads=8, kv_heads=1, ffn=4096,
                             dtype="bf16", mode="decode", batch=1, seq=16384),
}


class WeightSource:
    """Regenerates the weights of any (track, layer) on demand.

    ``get(t, l)`` returns a dict kind -> float32 array ([out, in] row-major for
    matrices), already rounded to bf16 when ``dtype == "bf16"``.  ``gain_jitter``
    > 0 replaces the all-ones norm gains by 1 + jitter*N(0,1) (used by tests so a
    missing gain multiply is visible); ``zero`` names kinds forced to zero.
    """

    def __init__(self, wl: Workload, seed: int | None = None, std: float = 0.02,
                 gain_jitter: float = 0.0, zero: tuple = (), router_std: float | None = None):
        self.wl, self.std, self.gain_jitter, self.zero = wl, std, gain_jitter, tuple(zero)
        self.router_std = std if router_std is None else router_std
        self.seed = wl.seed if seed is None else seed

    def one(self, t: int, l: int, kind: str) -> np.ndarray:
        shape = self.wl.weight_shape(kind)
        if kind in self.zero:
            return np.zeros(shape, np.float32)
        g = _rng(self.seed, _KIND_ID[kind], t, l)
        if kind in ("g1", "g2"):
            w = np.ones(shape, np.float32)
            if self.gain_jitter:
                w = w + np.float32(self.gain_jitter) * g.standard_normal(shape, dtype=np.float32)
        elif kind == "wr":
            return g.standard_normal(shape, dtype=np.float32) * np.float32(self.router_std)    # the router stays fp32
        else:
            w = g.standard_normal(shape, dtype=np.float32) * np.float32(self.std)
        return round_to_bf16(w) if self.wl.dtype == "bf16" else w

    def get(self, t: int, l: int) -> dict:
        return {k: self.one(t, l, k) for k in KINDS if k != "wr" or self.wl.experts}


def prefill_inputs(wl: Workload, batch: int | None = None, seq: int | None = None,
                   shared: bool = False, seed: int | None = None, salt: int = 0) -> np.ndarray:
    """Hidden-state inputs x[T, B, S, H] ~ N(0, 1), one independent draw per track
    (``shared`` = one draw broadcast to every track, Algorithm 1's literal case)."""
    B = wl.batch if batch is None else batch
    S = wl.seq if seq is None else seq
    seed = wl.seed if seed is None else seed
    out = np.empty((wl.T, B, S, wl.hidden), np.float32)
    for t in range(wl.T):
        src = 0 if shared else t
        out[t] = _rng(seed, _KIND_X, src, salt).standard_normal((B, S, wl.hidden), dtype=np.float32)
    return round_to_bf16(out) if wl.dtype == "bf16" else out


def decode_inputs(wl: Workload, batch: int | None = None, step: int = 0,
                  seed: int | None = None) -> np.ndarray:
    """New-token hidden states x[T, B, H] ~ N(0, 1) for decode step ``step``."""
    B = wl.batch if batch is None else batch
    seed = wl.seed if seed is None else seed
    out = np.empty((wl.T, B, wl.hidden), np.float32)
    for t in range(wl.T):
        out[t] = _rng(seed, _KIND_XDEC, t, step).standard_normal((B, wl.hidden), dtype=np.float32)
    return round_to_bf16(out) if wl.dtype == "bf16" else out


def kv_lengths(wl: Workload, batch: int | None = None, seed: int | None = None) -> np.ndarray:
    """KV length of every sequence BEFORE the decode step (int32[B]).
    Ragged workloads: integers uniform on [lo, hi], both ends included."""
    B = wl.batch if batch is None else batch
    seed = wl.seed if seed is None else seed
    if wl.ragged:
        lo, hi = wl.ragged
        full = _rng(seed, _KIND_LENS).integers(lo, hi + 1, wl.batch).astype(np.int32)
        return full[:B].copy()
    return np.full(B, wl.seq, np.int32)


def free_list_permutation(num_pages: int, seed: int = 0) -> np.ndarray:
    """A seeded permutation of page ids, used to make block tables non-monotonic."""
    return _rng(seed, _KIND_PERM).permutation(num_pages).astype(np.int32)
