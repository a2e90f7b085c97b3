"""CPU oracle for the Parallel Track (PT) transformer forward pass.  TEST INFRASTRUCTURE.

A plain, slow, float64 NumPy statement of what the PT forward computes, written
from the paper's Algorithm 1 ("Track Parallelism for PT Transformer", Section 2.2)
and the layer recipe of the workloads (pre-norm RMSNorm with eps inside the square
root, rotary embedding on half-split pairs, causal softmax attention with grouped
KV heads, SwiGLU feed-forward, no biases).  It exists only to check the CUDA path:
only tests, the smoke check and the CPU-baseline leg of the benchmark may import
it, and it shares no code with the CUDA path.

Every function below is pinned by the CPU tests to something other than itself
(closed forms, library routines, an independently written single-track decoder,
invariants of Algorithm 1, brute-force page enumeration); no function here is
"parity unpinned".  Declared conventions that nothing in the paper fixes (any
consistent choice is valid): rotary pairs are (j, j + dh/2); query head i reads
KV head i // G; the all-reduce of Algorithm 1 is a SUM (MEAN is available as an
option); "Set h_i = h" of Algorithm 1 is read as inside the if-block (its own
comment says it follows the all-reduce); the optional FP8 storage format of the KV
cache (E4M3 codes with one power-of-two scale per cached vector); the PT-MoE feed-forward
(linear router, top-k by logit with the lower index winning ties, softmax over the chosen logits).

Shapes: T tracks, L layers, D track-block depth, H per-track hidden, nq / nkv
query / KV heads per track, dh = H / nq, G = nq / nkv, F feed-forward width.
Weights are [out, in]; y = x @ W.T.  Positions are 0-based.
"""
from __future__ import annotations

from dataclasses import dataclass
import numpy as np


@dataclass(frozen=True)
class PTConfig:
    """Architecture numbers of a PT stack (Algorithm 1's n, L, D; Table 1's per-track heads)."""
    T: int
    D: int
    L: int
    hidden: int
    heads: int
    kv_heads: int
    ffn: int
    rope_base: float = 10000.0
    rms_eps: float = 1e-6
    sync_op: str = "sum"          # "sum" (the all-reduce of Algorithm 1) or "mean"
    experts: int = 0              # > 0: every track's feed-forward is a mixture of this many experts of width ffn (PT-MoE)
    top_k: int = 0                # experts evaluated per token

    def __post_init__(self):
        if self.T < 1 or self.L < 1 or self.D < 1:
            raise ValueError("T, L, D must be positive")
        if self.L % self.D:
            # Algorithm 1 returns the h of the last sync: trailing layers would be dropped.
            raise ValueError("L must be a multiple of D")
        if self.hidden % self.heads or self.heads % self.kv_heads:
            raise ValueError("hidden % heads and heads % kv_heads must be 0")
        if (self.hidden // self.heads) % 2:
            raise ValueError("head_dim must be even for rotary pairs")
        if self.sync_op not in ("sum", "mean"):
            raise ValueError("sync_op")
        if self.experts < 0 or (self.experts > 0 and not 1 <= self.top_k <= self.experts) or (self.experts == 0 and self.top_k):
            raise ValueError("top_k must lie in [1, experts]")

    @property
    def head_dim(self) -> int:
        return self.hidden // self.heads

    @property
    def group(self) -> int:
        return self.heads // self.kv_heads


def sync_points_pt(L: int, D: int) -> int:
    """Number of synchronisation points of a PT stack: one per track block (Section 2.2)."""
    return L // D


def sync_points_tp(L: int) -> int:
    """Tensor parallelism synchronises after attention and after the feed-forward
    of every layer (Section 2.1)."""
    return 2 * L


def sync_fraction_removed(L: int, D: int) -> float:
    """Share of tensor parallelism's sync points that PT removes (Section 2.2)."""
    return 1.0 - sync_points_pt(L, D) / sync_points_tp(L)


# ----------------------------------------------------------------------------- layer pieces

def rmsnorm(h: np.ndarray, g: np.ndarray, eps: float) -> np.ndarray:
    """h / sqrt(mean_k h_k^2 + eps) * g over the last axis."""
    ms = np.mean(h * h, axis=-1, keepdims=True)
    return h / np.sqrt(ms + eps) * g


def rope(u: np.ndarray, pos: np.ndarray, base: float) -> np.ndarray:
    """Rotate the pairs (j, j + dh/2) of u[..., S, heads, dh] by pos * base**(-2j/dh)."""
    dh = u.shape[-1]
    half = dh // 2
    j = np.arange(half, dtype=np.float64)
    theta = np.float64(base) ** (-2.0 * j / dh)
    ang = np.asarray(pos, np.float64)[:, None] * theta[None, :]        # [S, half]
    c = np.cos(ang)[:, None, :]
    s = np.sin(ang)[:, None, :]
    lo, hi = u[..., :half], u[..., half:]
    return np.concatenate([lo * c - hi * s, hi * c + lo * s], axis=-1)


def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def attention(q: np.ndarray, k: np.ndarray, v: np.ndarray, qpos: np.ndarray) -> np.ndarray:
    """Causal softmax attention for one sequence of one track.

    q [S, nq, dh] at absolute positions qpos[S]; k, v [N, nkv, dh] hold positions
    0..N-1.  Query head i reads KV head i // G and sees key j iff j <= qpos.
    Returns [S, nq, dh].
    """
    S, nq, dh = q.shape
    N, nkv, _ = k.shape
    G = nq // nkv
    out = np.empty_like(q)
    keypos = np.arange(N)
    visible = keypos[None, :] <= np.asarray(qpos)[:, None]             # [S, N]
    for i in range(nq):
        kh, vh = k[:, i // G, :], v[:, i // G, :]
        s = (q[:, i, :] @ kh.T) / np.sqrt(np.float64(dh))              # [S, N]
        s = np.where(visible, s, -np.inf)
        s = s - np.max(s, axis=-1, keepdims=True)
        p = np.exp(s)
        p = p / np.sum(p, axis=-1, keepdims=True)
        out[:, i, :] = p @ vh
    return out


def moe_gates(logits: np.ndarray, top_k: int) -> np.ndarray:
    """Routing weights of a mixture-of-experts layer: for every row of logits[..., E] the top_k largest
    logits (the lower index wins a tie) get softmax weights among themselves, all others 0."""
    logits = np.asarray(logits, np.float64)
    E = logits.shape[-1]
    # stable sort of -logits: equal logits keep index order, so the lower index ranks first
    order = np.argsort(-logits, axis=-1, kind="stable")
    chosen = order[..., :top_k]
    sel = np.take_along_axis(logits, chosen, axis=-1)
    w = np.exp(sel - sel.max(axis=-1, keepdims=True))
    w = w / w.sum(axis=-1, keepdims=True)
    gates = np.zeros(logits.shape)
    np.put_along_axis(gates, chosen, w, axis=-1)
    return gates


def moe_ffn(c: np.ndarray, wr: np.ndarray, wg: np.ndarray, wu: np.ndarray, wd: np.ndarray, top_k: int) -> np.ndarray:
    """PT-MoE feed-forward of one track (the paper names it in one sentence - an MoE layer inside each track -
    and defines nothing else; declared here): router logits c wr^T over E experts, moe_gates, and
    sum_e gate_e * (silu(c wg[e]^T) * (c wu[e]^T)) wd[e]^T.  wr [E, H], wg / wu [E, F, H], wd [E, H, F]."""
    gates = moe_gates(c @ wr.T, top_k)
    out = np.zeros(c.shape)
    for e in range(wr.shape[0]):
        y = (silu(c @ wg[e].T) * (c @ wu[e].T)) @ wd[e].T
        out = out + gates[..., e:e + 1] * y
    return out


# ----------------------------------------------------------------------------- FP8 KV-cache format
# Not in the paper (it has no cache at all): a declared storage format for K and V that halves the
# bytes of the cache, so that the ragged decode workload fits one device whole.  Every cached vector
# (one token, one KV head, head_dim values, K or V) is stored as E4M3 codes times one scale:
#   scale = the smallest power of two s >= 2^-100 with max|v| / s <= 448   (1 for an all-zero vector;
#           the floor keeps the scale a normal fp32 number whatever the vector holds)
#   code  = v / s rounded to the nearest E4M3 value, ties to the even mantissa, saturating at +-448
# E4M3 (the "FN" variant of the OCP 8-bit floating point formats): 1 sign, 4 exponent (bias 7) and 3
# mantissa bits; normal values (1 + m/8) * 2^(e-7) for e = 1..15 (the code e = 15, m = 7 is NaN, so the
# largest value is 1.75 * 2^8 = 448), subnormals (m/8) * 2^-6, no infinities.  Attention reads code * s.

E4M3_MAX = 448.0


def e4m3_round(x: np.ndarray) -> np.ndarray:
    """x (float64) -> the nearest E4M3 value, ties to even, saturating at +-448."""
    x = np.asarray(x, np.float64)
    a = np.minimum(np.abs(x), E4M3_MAX)
    with np.errstate(divide="ignore"):
        e = np.floor(np.log2(np.where(a > 0, a, 1.0)))
    e = np.maximum(e, -6.0)                        # below 2^-6 the spacing stays that of the subnormals
    step = np.exp2(e - 3.0)                        # 8 steps per binade
    q = np.rint(a / step) * step                   # numpy rounds halves to even; a carry into the next binade is exact
    return np.copysign(np.minimum(q, E4M3_MAX), x)


def kv_scale(v: np.ndarray) -> np.ndarray:
    """Power-of-two scale of each vector along the last axis (shape [..., 1])."""
    amax = np.max(np.abs(np.asarray(v, np.float64)), axis=-1, keepdims=True)
    with np.errstate(divide="ignore"):
        e = np.maximum(np.ceil(np.log2(np.where(amax > 0, amax, 1.0) / E4M3_MAX)), -100.0)
    return np.where(amax > 0, np.exp2(e), 1.0)


def kv_quantize(v: np.ndarray):
    """(codes, scale): codes are E4M3 values (as float64), scale [..., 1]; the cached value is codes * scale."""
    s = kv_scale(v)
    return e4m3_round(np.asarray(v, np.float64) / s), s


# ----------------------------------------------------------------------------- paged KV cache

def kv_slot_offset(cfg: PTConfig, num_pages: int, page_size: int,
                   t: int, l: int, page: int, kv: int, head: int, slot: int) -> int:
    """Element offset of the first of the dh values of one cached K (kv=0) or V (kv=1)
    vector in the pool laid out as [T][L][page][K|V][kv_head][slot][dh]."""
    return (((((t * cfg.L + l) * num_pages + page) * 2 + kv) * cfg.kv_heads + head)
            * page_size + slot) * cfg.head_dim


class PagedKVCache:
    """Per-track, per-layer paged KV cache with a host page allocator.

    The pool is one float64 array indexed exactly like ``kv_slot_offset``.  Pages
    are handed out from the front of a free list (ascending page ids unless
    ``free_order`` gives another order); one page id serves every (track, layer)
    slab of the pool.  ``block_table[seq][i]`` is the page holding positions
    i*page_size .. (i+1)*page_size-1 of sequence ``seq``.
    """

    def __init__(self, cfg: PTConfig, num_pages: int, page_size: int = 16, free_order=None, kv_format: str = "model"):
        if kv_format not in ("model", "e4m3"):
            raise ValueError("kv_format")
        self.cfg, self.num_pages, self.page_size, self.kv_format = cfg, num_pages, page_size, kv_format
        # what attention reads: the values themselves, or (kv_format "e4m3") code * scale of the FP8 format above
        self.pool = np.zeros((cfg.T, cfg.L, num_pages, 2, cfg.kv_heads, page_size, cfg.head_dim))
        # one scale per cached vector, indexed like the pool without its last axis (all ones for "model")
        self.scale = np.ones((cfg.T, cfg.L, num_pages, 2, cfg.kv_heads, page_size))
        order = list(range(num_pages)) if free_order is None else [int(p) for p in free_order]
        if sorted(order) != list(range(num_pages)):
            raise ValueError("free_order must be a permutation of the page ids")
        self.free = order
        self.block_table: dict[int, list[int]] = {}
        self.length: dict[int, int] = {}

    def reserve(self, seq: int, new_len: int) -> None:
        """Make room for positions < new_len of ``seq`` (does not change its length)."""
        table = self.block_table.setdefault(seq, [])
        self.length.setdefault(seq, 0)
        need = -(-new_len // self.page_size)
        if need - len(table) > len(self.free):
            raise MemoryError("KV cache full")
        while len(table) < need:
            table.append(self.free.pop(0))

    def release(self, seq: int) -> None:
        """Return a sequence's pages to the back of the free list, in table order."""
        self.free.extend(self.block_table.pop(seq, []))
        self.length.pop(seq, None)

    def locate(self, seq: int, pos: int) -> tuple[int, int]:
        return self.block_table[seq][pos // self.page_size], pos % self.page_size

    def _pages_slots(self, seq: int, pos: np.ndarray):
        pos = np.asarray(pos, np.int64)
        table = np.asarray(self.block_table[seq], np.int64)
        return table[pos // self.page_size], pos % self.page_size

    def write(self, t: int, l: int, seq: int, pos: np.ndarray, k: np.ndarray, v: np.ndarray) -> None:
        """Store k, v [n, nkv, dh] at positions pos[n] of ``seq``."""
        pages, slots = self._pages_slots(seq, pos)
        if self.kv_format == "e4m3":
            (kc, ks), (vc, vs) = kv_quantize(k), kv_quantize(v)
            k, v = kc * ks, vc * vs
            self.scale[t, l, pages, 0, :, slots] = ks[..., 0]
            self.scale[t, l, pages, 1, :, slots] = vs[..., 0]
        self.pool[t, l, pages, 0, :, slots, :] = k
        self.pool[t, l, pages, 1, :, slots, :] = v

    def gather(self, t: int, l: int, seq: int, n: int) -> tuple[np.ndarray, np.ndarray]:
        """K and V of positions 0..n-1 as [n, nkv, dh] each."""
        pages, slots = self._pages_slots(seq, np.arange(n))
        return self.pool[t, l, pages, 0, :, slots, :], self.pool[t, l, pages, 1, :, slots, :]


# ----------------------------------------------------------------------------- the PT forward

def _layer(cfg: PTConfig, w: dict, h: np.ndarray, cache: PagedKVCache, t: int, l: int,
           seq_ids, start, taps: dict | None) -> np.ndarray:
    """One standard pre-norm transformer layer of track t on h[B, S, H]."""
    B, S, H = h.shape
    nq, nkv, dh = cfg.heads, cfg.kv_heads, cfg.head_dim
    W = {k: np.asarray(a, np.float64) for k, a in w.items()}
    a = rmsnorm(h, W["g1"], cfg.rms_eps)
    q = (a @ W["wq"].T).reshape(B, S, nq, dh)
    k = (a @ W["wk"].T).reshape(B, S, nkv, dh)
    v = (a @ W["wv"].T).reshape(B, S, nkv, dh)
    o = np.empty((B, S, nq, dh))
    for b in range(B):
        pos = start[b] + np.arange(S)
        qb = rope(q[b], pos, cfg.rope_base)
        kb = rope(k[b], pos, cfg.rope_base)
        cache.write(t, l, seq_ids[b], pos, kb, v[b])
        kk, vv = cache.gather(t, l, seq_ids[b], start[b] + S)
        o[b] = attention(qb, kk, vv, pos)
    attn_delta = o.reshape(B, S, nq * dh) @ W["wo"].T
    h = h + attn_delta
    c = rmsnorm(h, W["g2"], cfg.rms_eps)
    if cfg.experts:
        ffn_delta = moe_ffn(c, W["wr"], W["wg"], W["wu"], W["wd"], cfg.top_k)
        if taps is not None:
            taps.setdefault("router_logits", {})[(t, l)] = c @ W["wr"].T
    else:
        ffn_delta = (silu(c @ W["wg"].T) * (c @ W["wu"].T)) @ W["wd"].T
    if taps is not None:
        taps.setdefault("attn_delta", {})[(t, l)] = attn_delta
        taps.setdefault("ffn_delta", {})[(t, l)] = ffn_delta
    return h + ffn_delta


def pt_prefill(cfg: PTConfig, weights, x: np.ndarray, cache: PagedKVCache, seq_ids,
               taps: dict | None = None) -> np.ndarray:
    """Algorithm 1 on x[T, B, S, H]; returns h[B, S, H].

    ``weights.get(t, l)`` gives the weight dict of track t, layer l (0-based).  The
    S tokens of batch row b are appended to sequence seq_ids[b] after the tokens it
    already holds.  ``x[t]`` is track t's starting state (Algorithm 1 uses the same
    x for every track; pass T equal slices for that case).  If ``taps`` is a dict it
    receives ``taps["h"][l]`` = the [T, B, S, H] residual stream after layer l
    (after the sync when l closes a track block) and the per-layer deltas.
    """
    x = np.asarray(x, np.float64)
    T, B, S, H = x.shape
    assert T == cfg.T and H == cfg.hidden and len(seq_ids) == B
    start = []
    for b in range(B):
        cache.reserve(seq_ids[b], cache.length.get(seq_ids[b], 0) + S)
        start.append(cache.length[seq_ids[b]])
    h = [x[t].copy() for t in range(T)]                       # Set h_i = x
    syncs = 0
    for l in range(cfg.L):                                    # for each layer
        for t in range(T):                                    # every track, independently
            h[t] = _layer(cfg, weights.get(t, l), h[t], cache, t, l, seq_ids, start, taps)
        if (l + 1) % cfg.D == 0:                              # one sync point per track block
            total = h[0].copy()
            for t in range(1, T):
                total = total + h[t]                          # all-reduce (sum)
            if cfg.sync_op == "mean":
                total = total / T
            h = [total.copy() for _ in range(T)]              # every track continues from h
            syncs += 1
        if taps is not None:
            taps.setdefault("h", {})[l] = np.stack(h)
    for b in range(B):
        cache.length[seq_ids[b]] = start[b] + S
    if taps is not None:
        taps["syncs"] = syncs
    assert syncs == sync_points_pt(cfg.L, cfg.D)
    return h[0]


def pt_decode_step(cfg: PTConfig, weights, x: np.ndarray, cache: PagedKVCache, seq_ids,
                   taps: dict | None = None) -> np.ndarray:
    """One new token per sequence: x[T, B, H] -> h[B, H].  The token of row b is
    written at position length[seq] and attends positions 0..length[seq]."""
    x = np.asarray(x, np.float64)
    return pt_prefill(cfg, weights, x[:, :, None, :], cache, seq_ids, taps)[:, 0, :]


# ----------------------------------------------------------------------------- ends of the model
# Algorithm 1 starts from the embedding output x and returns h; the paper measures time to first
# token and time per output token (Tables 6-10), which need the two ends it does not spell out.
# Declared conventions (nothing in the paper fixes them): one embedding table shared by all
# tracks (Algorithm 1's "Set h_i = x"), a final RMSNorm with its own gain on h, an untied
# LM-head matrix, greedy decoding that takes the lowest index among equal maxima.

def embed(table: np.ndarray, tokens: np.ndarray) -> np.ndarray:
    """Row tokens[...] of the embedding table [vocab, H] -> [..., H]."""
    return np.asarray(table, np.float64)[np.asarray(tokens, np.int64)]


def lm_head(h: np.ndarray, gain: np.ndarray, w_out: np.ndarray, eps: float) -> np.ndarray:
    """logits = rmsnorm(h; gain) @ w_out.T with w_out [vocab, H]."""
    return rmsnorm(np.asarray(h, np.float64), np.asarray(gain, np.float64), eps) @ np.asarray(w_out, np.float64).T


def greedy(logits: np.ndarray) -> np.ndarray:
    """Index of the largest logit per row (the lowest index when several are equal)."""
    return np.argmax(logits, axis=-1).astype(np.int64)


def pt_generate(cfg: PTConfig, weights, table, gain, w_out, prompt: np.ndarray, n_new: int,
                cache: PagedKVCache, seq_ids, round_x=None):
    """Greedy generation: prefill the prompt [B, S] (token ids), take the next token from the last
    position's logits, then one decode step per further token.  Every track starts from the same
    embedding (Algorithm 1).  ``round_x`` (optional) is applied to the embedded inputs, for callers
    whose model consumes them in a narrower type.  Returns (tokens [B, n_new], logits [B, n_new, V])."""
    prompt = np.asarray(prompt, np.int64)
    B, S = prompt.shape
    fix = round_x if round_x is not None else (lambda a: a)
    x = fix(embed(table, prompt))                                       # [B, S, H]
    h = pt_prefill(cfg, weights, np.broadcast_to(x, (cfg.T,) + x.shape), cache, seq_ids)
    out_tok = np.zeros((B, n_new), np.int64)
    out_logits = []
    logits = lm_head(h[:, -1, :], gain, w_out, cfg.rms_eps)              # [B, V]
    for i in range(n_new):
        out_logits.append(logits)
        out_tok[:, i] = greedy(logits)
        if i + 1 == n_new:
            break
        x = fix(embed(table, out_tok[:, i]))                              # [B, H]
        h = pt_decode_step(cfg, weights, np.broadcast_to(x, (cfg.T,) + x.shape), cache, seq_ids)
        logits = lm_head(h, gain, w_out, cfg.rms_eps)
    return out_tok, np.stack(out_logits, axis=1)
