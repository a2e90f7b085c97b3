"""The E4M3 storage format of the KV cache on the GPU, against the oracle's.

  * the quantiser alone, bit for bit: scale and codes of crafted and random bf16 vectors (the decision which
    code a value gets is taken on the same bf16 inputs on both sides);
  * whole forwards with an E4M3 cache (chunked prefill with earlier context, decode steps over several key
    ranges, GQA groups of 1, 4 and 8, pages of 16 and 32 tokens, shuffled pages) against the oracle with the
    same cache format: final output and every layer's stream within 2e-2 of the maximum and within the mean
    bound derived from the measured floor (tests/bf16_floor.py with kv8: the device quantises the K and V its
    bf16 GEMM produced, the oracle its exact ones, so a value near a code boundary lands one code step away;
    that, not bf16 rounding, sets the floor); scales and cached values; page tables bit-exact;
  * the two decode-attention kernels alone on caches the oracle quantised (both sides read the same codes and
    scales, so only the kernels' own arithmetic differs): random scores, scores that climb steadily or jump by
    2^5 / 2^7.5 after a key range's first tile (the running reference maximum and the range of the 8-bit
    probabilities), V magnitudes that double along the sequence, one to eight query heads per KV head.
"""
import functools

import numpy as np
import pytest

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I
from tests import helpers as Hp
from tests.test_gpu_parity import _check_taps

pytestmark = pytest.mark.gpu

# A layer's attention delta on its own scale feels the code flips directly (a flipped code is a sixteenth of its
# binade off, the delta averages some hundred of them): its max-error bound is widened from 2e-2 accordingly.
DELTA_TOL = 6e-2


def test_quantiser_matches_the_oracle_bit_for_bit():
    import torch
    from paper_2602_07306_b200 import pt
    rng = np.random.default_rng(0)
    n = 4096
    v = rng.standard_normal((n, 128)).astype(np.float32) * np.exp2(rng.integers(-30, 20, (n, 1))).astype(np.float32)
    v[0] = 0.0                                              # all zero: scale 1
    v[1] = 0.0; v[1, 7] = 448.0                             # the largest code at scale 1
    v[2] = 0.0; v[2, 7] = 450.0                             # mantissa above 1.75: the scale doubles
    v[3] = 0.0; v[3, 0] = 1.75; v[3, 1] = 1.0 / 512         # smallest subnormal code at scale 2^-8
    v[4] = 0.0; v[4, 3] = -3e-38                            # near the bottom of fp32: the scale's floor 2^-100
    v[5] = np.linspace(-448, 448, 128)                      # ties between codes
    v[6] = 0.0; v[6, 0] = 1e-41                             # a subnormal maximum
    v = I.round_to_bf16(v)
    codes, scales, status = pt.kernel_kv_quant_e4m3(torch.from_numpy(v).to("cuda:0").to(torch.bfloat16))
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0]
    want_codes, want_scale = O.kv_quantize(v.astype(np.float64))
    np.testing.assert_array_equal(scales.cpu().numpy().astype(np.float64), want_scale[:, 0])
    got = codes.view(torch.float8_e4m3fn).to(torch.float32).cpu().numpy().astype(np.float64)
    np.testing.assert_array_equal(got, want_codes)


def run_kv8_case(wl, *, B, chunks, decode_steps, ps=16, shuffle=True, sync_op="sum", flags=0):
    import torch
    ws = I.WeightSource(wl, gain_jitter=0.1)
    cfg = Hp.oracle_cfg(wl, sync_op)
    S = sum(chunks)
    total = S + decode_steps
    pages = B * (-(-total // ps)) + 2
    order = I.free_list_permutation(pages, seed=11) if shuffle else None
    seq_ids = [3 + 2 * b for b in range(B)]
    model = Hp.make_model(wl, ws, sync_op=sync_op, max_pos=max(64, total), flags=flags)
    cache = model.new_cache(pages, ps, order, kv_dtype="e4m3")
    cache.pool.zero_()
    ocache = O.PagedKVCache(cfg, pages, ps, order, kv_format="e4m3")
    mean_tol = Hp.mean_bound(wl, kv8=True)
    x = I.prefill_inputs(wl, batch=B, seq=S)
    s0, worst = 0, 0.0
    for n in chunks:
        xs = x[:, :, s0:s0 + n]
        taps = {}
        ref = O.pt_prefill(cfg, ws, xs, ocache, seq_ids, taps)
        tap = model.set_tap(-1, B * n)
        got = model.prefill(cache, Hp.to_dev(model, xs), seq_ids)
        torch.cuda.synchronize()
        assert model.device_status() == (0, 0)
        Hp.assert_close(got.cpu().numpy(), ref, wl.dtype, f"prefill chunk at {s0}", mean_tol=mean_tol,
                        log=f"e4m3 cache, {wl.name}: prefill chunk of {n} at {s0}")
        worst = max(worst, _check_taps(wl, tap.cpu().numpy(), taps, B, n, mean_tol, delta_tol=DELTA_TOL))
        s0 += n
    for step in range(decode_steps):
        xd = I.decode_inputs(wl, batch=B, step=step)
        taps = {}
        ref = O.pt_decode_step(cfg, ws, xd, ocache, seq_ids, taps)
        tap = model.set_tap(-1, B)
        got = model.decode_step(cache, Hp.to_dev(model, xd), seq_ids)
        torch.cuda.synchronize()
        assert model.device_status() == (0, 0)
        Hp.assert_close(got.cpu().numpy(), ref, wl.dtype, f"decode step {step}", mean_tol=mean_tol,
                        log=f"e4m3 cache, {wl.name}{' (mma.sync kernel)' if flags & 4 else ''}: decode step {step} at KV {S + step}")
        worst = max(worst, _check_taps(wl, tap.cpu().numpy(), taps, B, 1, mean_tol, delta_tol=DELTA_TOL))
    Hp.record(f"e4m3 cache, {wl.name}: largest error of a layer delta on its own scale", worst, float("nan"), DELTA_TOL, float("nan"))
    model.set_tap(None)
    for s in seq_ids:
        assert cache.block_table(s) == ocache.block_table[s]
        assert cache.length(s) == ocache.length[s] == total
    # the pool: scales are powers of two; where both sides chose the same scale the cached values differ by at most
    # one code step of that scale (a sixteenth of the vector's binade top); most vectors must have the same scale
    deq = cache.dequantized().cpu().numpy().astype(np.float64)
    scales = cache.scales.view(deq.shape[:-1]).cpu().numpy().astype(np.float64)
    written = np.zeros(deq.shape[:-1], bool)
    for s in seq_ids:
        for pos in range(total):
            page, slot = ocache.locate(s, pos)
            written[:, :, page, :, :, slot] = True
    sg, so = scales[written], ocache.scale[written]
    assert np.all(np.log2(sg) == np.round(np.log2(sg)))
    same = sg == so
    assert same.mean() > 0.97 and np.all((sg == so) | (sg == 2 * so) | (2 * sg == so))
    d = np.abs(deq[written] - ocache.pool[written])
    step_size = np.maximum(sg, so)[:, None] * 32.0           # the largest code step: 2^5 in units of the scale
    assert np.all(d <= step_size * (1 + 1e-6))
    mx, mean = Hp.rel_errs(deq[written], ocache.pool[written])
    Hp.record(f"e4m3 cache, {wl.name}: cached code * scale against the oracle's", mx, mean, 32.0 / 224.0, float("nan"))
    assert not np.any(deq[~written] != 0.0), "a slot outside the expected set was written"
    model.close()


def _wl(name, T, L, D, H, nq, nkv, F):
    return I.Workload(name, T=T, L=L, D=D, hidden=H, heads=nq, kv_heads=nkv, ffn=F, dtype="bf16", mode="prefill",
                      batch=1, seq=64, seed=0)


# Decode attention of an E4M3 cache has two kernels: the tcgen05 one (codes straight into 8-bit MMAs, keys on the M
# dimension; the default) and the mma.sync one (codes converted to f16; config flag bit 2).  Both run every case.
KERNELS = pytest.mark.parametrize("flags", [0, 4], ids=["tcgen05", "mma_sync"])


@KERNELS
def test_e4m3_cache_chunked_prefill_and_decode_mha(flags):
    run_kv8_case(_wl("kv8-mha", 2, 4, 2, 256, 2, 2, 352), B=3, chunks=[24, 1, 23], decode_steps=3, flags=flags)


@KERNELS
def test_e4m3_cache_gqa4_pages_of_32_tokens(flags):
    run_kv8_case(_wl("kv8-gqa4", 2, 2, 1, 512, 4, 1, 176), B=2, chunks=[40, 30], decode_steps=2, ps=32, flags=flags)


@KERNELS
def test_e4m3_cache_gqa8_long_sequences_split_over_key_ranges(flags):
    # 700 cached keys and few sequences: the decode step splits every sequence over several key ranges
    run_kv8_case(_wl("kv8-gqa8", 2, 2, 2, 1024, 8, 1, 256), B=2, chunks=[512, 188], decode_steps=2, sync_op="mean", flags=flags)


def _kv8_attention_case(T, B, nq, nkv, ps, lens, seed, climb_log2=0.0, climb_at=0, v_scale_steps=0):
    """A random paged E4M3 cache (quantised by the oracle) and bf16 queries; the float64 result of oracle.attention
    over code * scale.  With climb_log2 the first query head of every KV head sees scores that rise by that many
    powers of two along a sequence (keys aligned with the query, growing in length): steadily from the first key to
    the last, or, with climb_at, all at once at that key.  With v_scale_steps the magnitude of V doubles that many
    times along a sequence."""
    import torch
    rng = np.random.default_rng(seed)
    G, dh = nq // nkv, 128
    maxp = max(-(-int(n) // ps) for n in lens)
    pages = sum(-(-int(n) // ps) for n in lens) + 2
    perm = I.free_list_permutation(pages, seed=seed)
    bt = np.zeros((B, maxp), np.int32)
    nxt = 0
    for b, n in enumerate(lens):
        k = -(-int(n) // ps)
        bt[b, :k] = perm[nxt:nxt + k]
        nxt += k
    pool = rng.standard_normal((T, pages, 2, nkv, ps, dh))
    q = rng.standard_normal((T, B, nq, dh))
    if climb_log2 or v_scale_steps:
        beta = 10.0
        for t in range(T):
            for b, n in enumerate(lens):
                pos = np.arange(int(n))
                pg, sl = bt[b, pos // ps], pos % ps
                rise = (pos >= climb_at).astype(np.float64) if climb_at else pos / max(1, int(n) - 1)
                # a score in powers of two is log2(e) * beta * alpha / sqrt(dh)
                alpha = rise * climb_log2 * np.sqrt(dh) / (np.log2(np.e) * beta)
                for h in range(nkv):
                    if climb_log2:
                        u = rng.standard_normal(dh)
                        u /= np.linalg.norm(u)
                        q[t, b, h * G] = beta * u
                        pool[t, pg, 0, h, sl] = alpha[:, None] * u[None, :] + 0.3 * pool[t, pg, 0, h, sl]
                    if v_scale_steps:
                        pool[t, pg, 1, h, sl] *= np.exp2(np.floor(pos * v_scale_steps / int(n)))[:, None]
    q = I.round_to_bf16(q.astype(np.float32)).astype(np.float64)
    codes, scale = O.kv_quantize(pool.reshape(-1, dh))
    deq = (codes * scale).reshape(pool.shape)
    ref = np.zeros((T, B, nq * dh))
    for t in range(T):
        for b, n in enumerate(lens):
            pos = np.arange(int(n))
            k = deq[t, bt[b, pos // ps], 0, :, pos % ps, :]
            v = deq[t, bt[b, pos // ps], 1, :, pos % ps, :]
            ref[t, b] = O.attention(q[t, b].reshape(1, nq, dh), k, v, np.array([int(n) - 1])).reshape(-1)
    code_bytes = torch.from_numpy(codes.astype(np.float32)).to(torch.float8_e4m3fn).view(torch.uint8)
    dev = lambda a: a.to("cuda:0").contiguous()
    return (dev(torch.from_numpy(q.reshape(T, B, nq * dh).astype(np.float32)).to(torch.bfloat16)),
            dev(code_bytes.reshape(T, pages, 2, nkv, ps, dh)),
            dev(torch.from_numpy(scale.reshape(T, pages, 2, nkv, ps).astype(np.float32))),
            dev(torch.from_numpy(bt)), ref)


@functools.lru_cache(maxsize=1)
def _cached_case(T, B, nq, nkv, ps, lens, seed, climb, at, vsteps):
    return _kv8_attention_case(T, B, nq, nkv, ps, list(lens), seed, climb_log2=climb, climb_at=at, v_scale_steps=vsteps)


# The kernels keep q and the probabilities as pairs of E4M3 numbers (relative error 2^-8 per element) and write bf16.
ATTN8_MAX, ATTN8_MEAN = 1e-2, 3e-3

# With many sequences a key range is a whole sequence (the planner splits only to fill the machine), so one CTA walks
# all of a sequence's tiles with one running reference maximum.
MANY = 80


@pytest.mark.parametrize("impl", [0, 1], ids=["tcgen05", "mma_sync"])
@pytest.mark.parametrize("T,B,nq,nkv,ps,lens,climb,at,vsteps", [
    (2, 3, 8, 2, 16, [1, 130, 700], 0.0, 0, 0),                 # random scores; one key, a tile and a bit, several tiles and ranges
    (1, 2, 4, 1, 16, [2048, 700], 14.0, 0, 0),                  # a steady climb by 2^14 over many short key ranges
    (1, 2, 8, 8, 32, [1500, 4097], 6.0, 0, 5),                  # one query head per KV head, V magnitudes double five times
    (2, 1, 8, 1, 16, [3000], 30.0, 0, 0),                       # a steep climb (2^30): early keys underflow, eight heads per KV head
    (2, MANY, 4, 2, 16, [384] * MANY, 5.0, 128, 0),             # the scores rise by 2^5 after the first tile and stay there: a reference
                                                                # maximum that is not raised at once leaves probabilities of 32 for most keys
    (2, MANY, 4, 2, 16, [400 + 3 * i for i in range(MANY)], 7.5, 200, 3),   # the same with 2^7.5 in mid-tile, ragged lengths, growing V
    (1, 2, 4, 2, 16, [900, 300], 0.0, 0, 24),                   # V magnitudes from 1 to 2^24 along a sequence: scales far apart in one tile's product
    (4, MANY, 4, 4, 16, [16 + (37 * i) % 190 for i in range(MANY - 2)] + [1200, 900], 3.0, 0, 2),   # a full machine without splits:
                                                                # only the two sequences far above the mean length get several key ranges
], ids=["random", "climb14", "climb6_v32", "climb30", "step5", "step7.5_v8", "v_2^24", "full_machine"])
def test_e4m3_decode_attention_kernels_against_the_oracle(impl, T, B, nq, nkv, ps, lens, climb, at, vsteps):
    import torch
    from paper_2602_07306_b200 import pt
    q, codes, scales, bt, ref = _cached_case(T, B, nq, nkv, ps, tuple(lens), len(lens) + nq, climb, at, vsteps)   # both kernels: the same case
    out, status = pt.kernel_decode_attn_e4m3(q, codes, scales, bt, lens, nq=nq, nkv=nkv, ps=ps, impl=impl)
    torch.cuda.synchronize()
    assert status[:2].tolist() == [0, 0]
    got = out.float().cpu().numpy().astype(np.float64)
    mx, mean = Hp.rel_errs(got, ref)
    Hp.record(f"e4m3 decode attention kernel ({'mma.sync' if impl else 'tcgen05'}), scores rising by 2^{climb:g}, {B} sequences of up to {max(lens)} keys",
              mx, mean, ATTN8_MAX, ATTN8_MEAN)
    assert mx <= ATTN8_MAX and mean <= ATTN8_MEAN, f"max-rel {mx:.3e}, mean-rel {mean:.3e}"
