"""Kernel-level parity through the C ABI: the tcgen05 track-grouped GEMM against the plain
definition sum_k a[t,m,k] w[t,n,k] evaluated in float64 from the same bf16-rounded operands."""
import numpy as np
import pytest

from paper_2602_07306_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _operands(T, M, N, K, seed):
    rng = np.random.default_rng(seed)
    a = I.round_to_bf16(rng.standard_normal((T, M, K), dtype=np.float32))
    w = I.round_to_bf16(rng.standard_normal((T, N, K), dtype=np.float32) * 0.05)
    return a, w


@pytest.mark.parametrize("T,M,N,K,bn,fold", [
    (1, 128, 128, 64, 128, False),        # one tile, one k-block
    (1, 128, 256, 256, 256, False),       # wide tile
    (2, 200, 384, 320, 128, False),       # ragged M, several tiles, tracks in the grid
    (3, 64, 2752, 128, 128, False),       # N tail (2752 = 21.5 x 128), M smaller than a tile
    (2, 300, 128, 1376, 128, False),      # K tail (1376 = 21.5 x 64)
    (4, 130, 512, 1376, 256, True),       # tracks folded into K (track-sync contraction)
    (2, 1024, 1024, 1024, 0, False),      # enough tiles for several per CTA, library-chosen width
    (3, 64, 1024, 320, 64, False),        # narrow tiles (decode shapes), few rows
    (2, 200, 160, 192, 64, True),         # narrow tiles, N tail, tracks folded into K
    (2, 1, 512, 1024, 64, False),         # one row: ring stages of 4 k-blocks, W copied 4 k-blocks at a time
    (1, 8, 192, 2048, 64, False),         # 8 stages' worth of k-blocks per tile: the ring wraps inside a tile
    (2, 64, 384, 768, 128, False),        # stages of 2 k-blocks
    (2, 176, 256, 512, 64, False),        # two row tiles, stages of 2 k-blocks
    (1, 40, 96, 256, 64, False),          # N tail inside a 4-k-block copy, one stage per tile
    (1, 16, 48, 256, 64, False),          # N smaller than the tile: the W box is 48 rows
    (2, 3, 640, 1024, 0, False),          # library-chosen width and stage shape at decode size
    (2, 1024, 512, 256, 256, False),      # CTA pairs on 256 x 256 tiles: full tiles, tracks in the grid
    (1, 1100, 640, 320, 256, False),      # CTA pairs: ragged M (the odd CTA's last rows are past M), N tail of half a tile
    (1, 1300, 256, 1376, 256, False),     # CTA pairs: last row tile has no rows for the odd CTA; K tail
    (3, 1024, 256, 192, 256, True),       # CTA pairs with tracks folded into K
    (1, 4096, 1024, 1024, 256, False),    # CTA pairs: more tiles than pairs, both accumulators in use
    (2, 176, 768, 512, 0, False),         # a large decode batch: one 256-row pair tile whose odd CTA holds 48 rows
    (3, 130, 256, 320, 0, False),         # the odd CTA holds two rows
    (4, 176, 3072, 2048, 0, False),       # CTA pairs at decode size (a 176-row batch against a wide projection): the ring wraps five times
    (2, 256, 5120, 384, 0, False),        # CTA pairs at decode size: exactly 256 rows, as many k-blocks as ring stages
    (2, 300, 2816, 320, 0, False),        # CTA pairs at decode size: two 256-row tiles, the second with 44 rows in its even CTA only
    (1, 512, 10368, 256, 0, False),       # CTA pairs at decode size: more tiles than pairs, N tail of half a tile
])
def test_gemm_bf16_matches_definition(T, M, N, K, bn, fold):
    import torch
    from paper_2602_07306_b200 import pt
    a, w = _operands(T, M, N, K, seed=M + N + K)
    ref = np.einsum("tmk,tnk->tmn", a.astype(np.float64), w.astype(np.float64))
    if fold:
        ref = ref.sum(0, keepdims=True)
    da = torch.from_numpy(a).cuda().to(torch.bfloat16)
    dw = torch.from_numpy(w).cuda().to(torch.bfloat16)
    c, status = pt.kernel_gemm_bf16(da, dw, bn=bn, fold_tracks=fold)
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0]
    got = c.cpu().numpy().astype(np.float64)
    err = np.abs(got - ref).max() / np.abs(ref).max()
    assert err <= 2e-6 * np.sqrt(K * (T if fold else 1)), f"max-rel {err:.3e}"     # fp32 accumulation of exact bf16 products


def _climbing_scores(rng, pool, q_rows, bt, b, t, n, nq, nkv, dh, ps, climb, at):
    """Rewrites the keys of sequence b (positions 0..n-1) and the first query head of every KV head (rows q_rows of
    q[t], shaped [rows, nq, dh]) so that the scores rise by `climb` powers of two along the sequence: keys and queries
    share a direction, the keys' length grows steadily from the first key to the last or, with `at`, all at once at
    that key.  A kernel that carries a running maximum has to raise it again and again (or once, late)."""
    G = nq // nkv
    pos = np.arange(n)
    pg, sl = bt[b, pos // ps], pos % ps
    rise = (pos >= at).astype(np.float64) if at else pos / max(1, n - 1)
    beta = 10.0
    alpha = rise * climb * np.sqrt(dh) / (np.log2(np.e) * beta)          # a score in powers of two: log2(e) beta alpha / sqrt(dh)
    for h in range(nkv):
        u = rng.standard_normal(dh)
        u /= np.linalg.norm(u)
        q_rows[:, h * G, :] = beta * u[None, :] + 0.1 * q_rows[:, h * G, :]
        pool[t, pg, 0, h, sl] = alpha[:, None] * u[None, :] + 0.3 * pool[t, pg, 0, h, sl]


def decode_case(T, B, nq, nkv, dh, ps, lens, seed, climb=0.0, at=0):
    """Random paged cache + queries; returns torch inputs and the float64 oracle result
    (oracle.attention on the gathered keys, one sequence and track at a time)."""
    import torch
    from oracle import pt_oracle as O
    rng = np.random.default_rng(seed)
    maxp = max(-(-int(n) // ps) for n in lens)
    pages = sum(-(-int(n) // ps) for n in lens) + 2
    perm = I.free_list_permutation(pages, seed=seed)
    bt = np.zeros((B, maxp), np.int32)
    nxt = 0
    for b, n in enumerate(lens):
        k = -(-int(n) // ps)
        bt[b, :k] = perm[nxt:nxt + k]
        nxt += k
    pool = rng.standard_normal((T, pages, 2, nkv, ps, dh), dtype=np.float32)
    q = rng.standard_normal((T, B, nq * dh), dtype=np.float32)
    if climb:
        for t in range(T):
            for b, n in enumerate(lens):
                _climbing_scores(rng, pool, q[t, b:b + 1].reshape(1, nq, dh), bt, b, t, int(n), nq, nkv, dh, ps, climb, at)
    pool, q = I.round_to_bf16(pool), I.round_to_bf16(q)
    ref = np.zeros((T, B, nq * dh))
    for t in range(T):
        for b, n in enumerate(lens):
            pos = np.arange(int(n))
            k = pool[t, bt[b, pos // ps], 0, :, pos % ps, :].astype(np.float64)       # [n, nkv, dh]
            v = pool[t, bt[b, pos // ps], 1, :, pos % ps, :].astype(np.float64)
            o = O.attention(q[t, b].reshape(1, nq, dh).astype(np.float64), k, v, np.array([int(n) - 1]))
            ref[t, b] = o.reshape(-1)
    dev = lambda a, dt: torch.from_numpy(a).cuda().to(dt).contiguous()
    return dev(q, torch.bfloat16), dev(pool, torch.bfloat16), dev(bt, torch.int32), ref


@pytest.mark.parametrize("T,B,nq,nkv,dh,ps,lens,climb,at", [
    (2, 3, 2, 2, 128, 16, [1, 17, 64], 0, 0),                 # single token, page tails, exactly one tile
    (1, 2, 8, 2, 64, 16, [300, 1023], 0, 0),                  # GQA 4:1, several key ranges per sequence
    (2, 4, 4, 1, 128, 16, [513, 4097, 2048, 15], 0, 0),       # ragged, long, GQA 4:1
    (1, 2, 4, 4, 32, 8, [100, 37], 0, 0),                     # small heads, 8-token pages
    (3, 2, 16, 2, 128, 32, [700, 90], 0, 0),                  # GQA 8:1, 32-token pages
    (1, 2, 8, 2, 128, 16, [2048, 700], 14.0, 0),              # scores climbing by 2^14 along the sequence: the running maximum rises in every tile
    (2, 80, 4, 2, 128, 16, [384] * 80, 7.5, 128),             # many sequences (one key range each): the scores jump by 2^7.5 after the first tile
    (1, 1, 4, 1, 64, 16, [3000], 60.0, 0),                    # a climb by 2^60: the early keys' weights underflow
    (4, 80, 4, 4, 64, 16, [16 + (37 * i) % 380 for i in range(77)] + [1500, 1100, 900], 0, 0),   # enough (sequence, track, KV head)
                                                              # triples to fill the machine: only the sequences far above the mean length are split
])
def test_decode_attention_kernel_matches_oracle(T, B, nq, nkv, dh, ps, lens, climb, at):
    import torch
    from paper_2602_07306_b200 import pt
    q, pool, bt, ref = decode_case(T, B, nq, nkv, dh, ps, lens, seed=sum(lens), climb=climb, at=at)
    out, status = pt.kernel_decode_attn(q, pool, bt, lens, nq=nq, nkv=nkv, dh=dh, ps=ps)
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0]
    got = out.float().cpu().numpy().astype(np.float64)
    d = np.abs(got - ref)
    assert d.max() <= 2e-2 * np.abs(ref).max() and d.mean() <= 4e-3 * np.abs(ref).mean(), (d.max() / np.abs(ref).max(), d.mean() / np.abs(ref).mean())


def test_decode_attention_kernel_reports_bad_page():
    """A page id outside the pool is skipped and reported through the status word (no fault)."""
    import torch
    from paper_2602_07306_b200 import pt
    q, pool, bt, _ = decode_case(1, 2, 2, 2, 64, 16, [40, 20], seed=3)
    bt[1, 0] = pool.shape[1] + 5
    out, status = pt.kernel_decode_attn(q, pool, bt, [40, 20], nq=2, nkv=2, dh=64, ps=16)
    torch.cuda.synchronize()
    assert status[0].item() == 8 and status[1].item() == 7
    assert torch.isfinite(out.float()).all()


def prefill_case(T, B, S, nq, nkv, dh, ps, starts, seed, climb=0.0, at=0):
    """Random paged cache holding starts[b] + S keys per sequence (slots past a sequence's last
    key hold NaN: they must never reach a result) + queries for the last S positions; the
    float64 result comes from oracle.attention, one sequence and track at a time."""
    import torch
    from oracle import pt_oracle as O
    rng = np.random.default_rng(seed)
    lens = [int(s0) + S for s0 in starts]
    maxp = max(-(-n // ps) for n in lens)
    pages = sum(-(-n // ps) for n in lens) + 2
    perm = I.free_list_permutation(pages, seed=seed)
    bt = np.zeros((B, maxp), np.int32)
    nxt = 0
    for b, n in enumerate(lens):
        k = -(-n // ps)
        bt[b, :k] = perm[nxt:nxt + k]
        nxt += k
    pool = rng.standard_normal((T, pages, 2, nkv, ps, dh), dtype=np.float32)
    q = rng.standard_normal((T, B * S, nq * dh), dtype=np.float32)
    if climb:
        for t in range(T):
            for b, n in enumerate(lens):
                _climbing_scores(rng, pool, q[t, b * S:(b + 1) * S].reshape(S, nq, dh), bt, b, t, n, nq, nkv, dh, ps, climb, at)
    pool, q = I.round_to_bf16(pool), I.round_to_bf16(q)
    ref = np.zeros((T, B * S, nq * dh))
    valid = np.zeros((pages, ps), bool)
    for t in range(T):
        for b, n in enumerate(lens):
            pos = np.arange(n)
            valid[bt[b, pos // ps], pos % ps] = True
            k = pool[t, bt[b, pos // ps], 0, :, pos % ps, :].astype(np.float64)
            v = pool[t, bt[b, pos // ps], 1, :, pos % ps, :].astype(np.float64)
            qb = q[t, b * S:(b + 1) * S].reshape(S, nq, dh).astype(np.float64)
            ref[t, b * S:(b + 1) * S] = O.attention(qb, k, v, starts[b] + np.arange(S)).reshape(S, -1)
    pool = np.where(valid[None, :, None, None, :, None], pool, np.float32(np.nan))
    dev = lambda a, dt: torch.from_numpy(a).cuda().to(dt).contiguous()
    return (dev(q, torch.bfloat16), dev(pool, torch.bfloat16), dev(bt, torch.int32),
            dev(np.asarray(lens, np.int32), torch.int32), ref)


PREFILL_CASES = [
    (1, 1, 128, 1, 1, 128, 16, [0]),                 # one query tile, one key tile
    (1, 1, 256, 2, 2, 128, 16, [0]),                 # both query tiles of a CTA, 1 and 2 key tiles
    (2, 2, 300, 4, 2, 128, 16, [0, 213]),            # ragged tails, earlier keys in the cache (chunked prefill), GQA 2:1
    (1, 3, 37, 2, 1, 64, 16, [0, 5, 100]),           # short chunks, head_dim 64
    (1, 2, 700, 2, 2, 64, 32, [513, 0]),             # 32-token pages, several CTAs per sequence
    (2, 1, 1024, 2, 1, 128, 16, [0]),                # keys end exactly on a tile boundary
    (1, 2, 1, 2, 2, 128, 16, [130, 0]),              # single new token per sequence
    (1, 1, 1024, 2, 1, 128, 16, [0], 40.0, 0),       # scores climbing by 2^40 along the keys: every row's maximum keeps rising, tile after tile
    (1, 2, 512, 2, 2, 128, 16, [300, 0], 7.5, 200),  # the scores jump by 2^7.5 at key 200: below the threshold at which the tensor-core kernel raises its reference
    (1, 2, 512, 4, 2, 128, 16, [0, 130], 9.0, 330),  # ... and above it, in mid-tile
    (1, 1, 700, 2, 2, 64, 32, [513], 20.0, 0),       # a climb over earlier context, head_dim 64, 32-token pages
]


@pytest.mark.parametrize("impl", [0, 1])
@pytest.mark.parametrize("case", PREFILL_CASES, ids=[f"S{c[2]}-dh{c[5]}-start{max(c[7])}" + (f"-climb{c[8]:g}" if len(c) > 8 else "") for c in PREFILL_CASES])
def test_prefill_attention_kernel_matches_oracle(case, impl):
    import torch
    from paper_2602_07306_b200 import pt
    T, B, S, nq, nkv, dh, ps, starts = case[:8]
    climb, at = (case[8], case[9]) if len(case) > 8 else (0.0, 0)
    q, pool, bt, lens, ref = prefill_case(T, B, S, nq, nkv, dh, ps, starts, seed=S + sum(starts), climb=climb, at=at)
    out, status = pt.kernel_prefill_attn(q, pool, bt, lens, S=S, nq=nq, nkv=nkv, dh=dh, ps=ps, impl=impl)
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0]
    got = out.float().cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(got))
    d = np.abs(got - ref)
    assert d.max() <= 2e-2 * np.abs(ref).max() and d.mean() <= 4e-3 * np.abs(ref).mean(), (d.max() / np.abs(ref).max(), d.mean() / np.abs(ref).mean())


def test_a_wait_that_nothing_ends_gives_up_in_time_and_leaves_the_context_usable():
    """The library's device-side waits are bounded in time: the self-test waits on a barrier at which nothing
    arrives, must come back after its limit with PT_ERR_DEVICE_TIMEOUT in the status block, and the next launch
    on the same context must still work (no trap, no fault, no endless spin)."""
    import time
    import torch
    from paper_2602_07306_b200 import pt
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    status = pt.kernel_wait_selftest(20_000_000)             # 20 ms
    torch.cuda.synchronize()
    dt = time.perf_counter() - t0
    assert status[:2].tolist() == [9, 20], status[:4].tolist()      # PT_ERR_DEVICE_TIMEOUT, the self-test's location code
    assert 0.015 <= dt < 1.0, dt
    with pytest.raises(pt.PtError):
        pt.kernel_wait_selftest(10)                          # below the accepted range: refused on the host
    a, w = _operands(1, 64, 64, 64, seed=1)
    c, st = pt.kernel_gemm_bf16(torch.from_numpy(a).cuda().to(torch.bfloat16), torch.from_numpy(w).cuda().to(torch.bfloat16))
    torch.cuda.synchronize()
    assert st[:2].tolist() == [0, 0]
    ref = np.einsum("tmk,tnk->tmn", a.astype(np.float64), w.astype(np.float64))
    assert np.abs(c.cpu().numpy() - ref).max() <= 1e-4 * np.abs(ref).max() + 1e-6
