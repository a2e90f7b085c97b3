"""Parity with the float64 oracle at the full sizes of the decode and prefill workloads, in the launch
configuration the benchmark times, at full depth, with the seeded NumPy weights.

The CPU oracle cannot run these workloads whole, so each is tied to it through outputs the oracle can
compute one by one:

  * prefill (T=8, L=32, 8 x 4096 tokens): causal attention makes the outputs of the first n tokens of a
    batch row depend on those n tokens only, so the oracle runs n = 400 tokens of two sampled rows alone
    (more than one 256-row query block, four 128-key tiles) and its result is compared with the same
    positions of the full-size launch: final output, cached K/V, and - in every track block - one layer's
    per-track stream and its attention and feed-forward deltas on their own scale (with SUM syncs the
    stream grows by about T per block, so a late block's work is invisible in the final output);
  * decode (batch 64 at KV 2048; the ragged GQA batch of the wide model): batch rows are independent, so
    the oracle follows sampled sequences of the full-size batch.  One sequence per workload is the
    oracle's from the first prompt token on ("own cache": it prefills the same seeded prompt itself); a
    second one starts from the K/V the device cached for it ("device cache": the pool slabs of that
    sequence are downloaded into the oracle's cache, which isolates the decode step at a length the
    oracle could not prefill in minutes).  For those rows the decode output, every layer's stream and both
    deltas are compared; for the own-cache sequence also the cached K/V.

Every comparison prints its measured errors (and appends them to the file PT_PARITY_LOG names, if set).
Mean bounds: helpers.mean_bound - 2e-3 where the arithmetic allows it, else the measured bf16-operand
floor times the stated margin.
"""
import numpy as np
import pytest

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I
from tests import helpers as Hp
from tests.test_gpu_parity import _check_taps

pytestmark = pytest.mark.gpu


def _free_gib():
    import torch
    return torch.cuda.mem_get_info()[0] / 2**30


@pytest.fixture(scope="module")
def mid_model():
    """The T=8, L=32 model shared by the batched-decode and long-prefill workloads, with the
    workloads' seeded weights (NumPy recipe, so the oracle can regenerate any (track, layer))."""
    wl = I.WORKLOADS["cfg3"]
    ws = I.WeightSource(wl)
    m = Hp.make_model(wl, Hp.Prefetch(ws, wl.T, wl.L), max_pos=4096)
    yield wl, ws, m
    m.close()


def _tap_layers(wl):
    """One layer per track block, at a different depth in each, never the block's last layer (its
    after-layer tap is the synced stream, which hides the feed-forward delta)."""
    return [k * wl.D + min(max(wl.D - 2, 0), 2 + k) for k in range(wl.L // wl.D)]


def test_prefill_full_size_sampled_prefixes_match_oracle(mid_model):
    import torch
    wl, ws, model = mid_model
    B, S, ps, T, H = wl.batch, wl.seq, wl.page_size, wl.T, wl.hidden
    if _free_gib() < 60:
        pytest.skip("needs about 60 GiB of free device memory")
    mean_tol = Hp.mean_bound(wl)
    pages = B * (S // ps)
    order = I.free_list_permutation(pages, seed=3)
    cache = model.new_cache(pages, ps, order)
    g = torch.Generator(device="cpu").manual_seed(1234)
    # inputs N(0, 1) rounded to bf16; the sampled rows are drawn with the NumPy recipe so the oracle sees the same values
    rows, n = [5, 2], 400                                  # sampled batch rows and the prefix length the oracle runs
    x = torch.randn((T, B, S, H), generator=g, dtype=torch.float32).to(torch.bfloat16)
    xs = I.prefill_inputs(wl, batch=len(rows), seq=n, salt=100)              # [T, 2, n, H], bf16-rounded NumPy draws
    for i, b in enumerate(rows):
        x[:, b, :n] = torch.from_numpy(xs[:, i]).to(torch.bfloat16)
    xdev = x.to(model.device)
    seq_ids = [11 + 2 * b for b in range(B)]

    cfg = Hp.oracle_cfg(wl)
    ocache = O.PagedKVCache(cfg, len(rows) * (-(-n // ps)), ps)
    taps = {}
    ref = O.pt_prefill(cfg, Hp.Prefetch(ws, T, wl.L), xs, ocache, list(range(len(rows))), taps)    # [2, n, H]

    def run(tap_layer):
        for s in seq_ids:
            cache.truncate(s, 0) if cache.length(s) else None
        tap = model.set_tap(tap_layer, B * S)
        got = model.prefill(cache, xdev, seq_ids)
        torch.cuda.synchronize()
        assert model.device_status() == (0, 0)
        sel = torch.cat([torch.arange(b * S, b * S + n) for b in rows]).to(model.device)
        t = tap[0][:, :, sel].cpu().numpy().astype(np.float64).reshape(2, T, len(rows), n, H)
        model.set_tap(None)
        return got, t

    got = None
    for l in _tap_layers(wl):
        # the stream entering layer l (end of layer l-1), then layer l's two tap points
        prev = np.stack([xs[t].astype(np.float64) for t in range(T)]) if l == 0 else run(l - 1)[1][1]
        got, tl = run(l)
        want_end = taps["h"][l]                                                                 # [T, 2, n, H]
        want_attn = np.stack([taps["h"][l - 1][t] if l else xs[t].astype(np.float64) for t in range(T)]) \
            + np.stack([taps["attn_delta"][(t, l)] for t in range(T)])
        Hp.assert_close(tl[0], want_attn, wl.dtype, f"layer {l}: per-track stream after attention", mean_tol=mean_tol,
                        log=f"cfg3 prefill 8x4096, rows {rows} x {n} tokens: layer {l} stream after attention")
        Hp.assert_close(tl[1], want_end, wl.dtype, f"layer {l}: per-track stream after the layer", mean_tol=mean_tol,
                        log=f"cfg3 prefill 8x4096, rows {rows} x {n} tokens: layer {l} stream after the layer")
        for t in range(T):
            # deltas on their own scale; the difference of two fp32 streams carries their rounding: allow it explicitly
            for name, gd, wd, base in (("attention", tl[0][t] - prev[t], taps["attn_delta"][(t, l)], prev[t]),
                                       ("ffn", tl[1][t] - tl[0][t], taps["ffn_delta"][(t, l)], tl[0][t])):
                mx, mean = Hp.rel_errs(gd, wd)
                slack = 4 * 6e-8 * np.abs(base).max() / max(np.abs(wd).max(), 1e-30)
                if t == 0:
                    Hp.record(f"cfg3 prefill 8x4096: layer {l} track 0 {name} delta (slack {slack:.1e})", mx, mean, 2e-2 + slack, float("nan"))
                assert mx <= 2e-2 + slack, f"layer {l} track {t} {name} delta: max-rel {mx:.3e}"
    for i, b in enumerate(rows):
        Hp.assert_close(got[b, :n].cpu().numpy(), ref[i], wl.dtype, f"row {b}: final output of the first {n} tokens",
                        mean_tol=mean_tol, log=f"cfg3 prefill 8x4096: final output, row {b}, first {n} tokens")
        # cached K/V of sampled positions in the first and last layer, through the library's own slot arithmetic
        pool = cache.pool
        for l in (0, wl.L - 1):
            for t in (0, T - 1):
                for pos in (0, 127, 128, n // 2, 255, 256, n - 1):
                    for kv in (0, 1):
                        off = cache.slot(t, l, seq_ids[b], pos, kv, 3)
                        dev = pool[off:off + wl.head_dim].float().cpu().numpy()
                        page, slot = ocache.locate(i, pos)
                        want = ocache.pool[t, l, page, kv, 3, slot]
                        d = np.abs(dev - want)
                        assert d.max() <= 2e-2 * np.abs(want).max() + 1e-6, f"row {b} layer {l} track {t} pos {pos} kv {kv}"
    cache.close()
    del cache, x, xdev
    torch.cuda.empty_cache()


def _seq_kv(cache, wl, t, pages):
    """What attention reads for track t on the given pages (a CUDA index tensor), all layers:
    float32 numpy [L, pages, K|V, head, slot, dh] - the cached values, or code * scale of an E4M3 cache -
    and the scales [L, pages, K|V, head, slot] (None for a cache in the model dtype)."""
    import torch
    shape = (wl.T, wl.L, cache.num_pages, 2, wl.kv_heads, wl.page_size)
    if cache.kv_dtype:
        codes = cache.codes.view(shape + (wl.head_dim,))[t][:, pages].view(torch.float8_e4m3fn).to(torch.float32)
        sc = cache.scales.view(shape)[t][:, pages]
        return (codes * sc.unsqueeze(-1)).cpu().numpy(), sc.cpu().numpy()
    return cache.pool.view(shape + (wl.head_dim,))[t][:, pages].float().cpu().numpy(), None


def _inject(cache, wl, seq, n, ocache, oseq):
    """Copy the first n cached tokens of device sequence `seq` into sequence `oseq` of the oracle's cache."""
    import torch
    ocache.reserve(oseq, n)
    ocache.length[oseq] = n
    pages = torch.tensor(cache.block_table(seq)[: -(-n // wl.page_size)], device=cache.pool.device)
    opages = np.asarray(ocache.block_table[oseq])
    for t in range(wl.T):
        blk, sc = _seq_kv(cache, wl, t, pages)                         # [L, pages, K|V, head, slot, dh]
        if n % wl.page_size:
            blk[:, -1, :, :, n % wl.page_size:, :] = 0.0               # slots past the sequence's end were never written
        ocache.pool[t][:, opages] = blk
        if sc is not None:
            if n % wl.page_size:
                sc[:, -1, :, :, n % wl.page_size:] = 1.0
            ocache.scale[t][:, opages] = sc


def _fill_and_decode(model, wl, lens, own, x_own, rows, xd_rows, seed, sub_tokens=16384, kv8=False):
    """Fill the cache of a full-size batch by prefills of N(0, 1) prompts (sequence `own` gets the NumPy-drawn
    prompt x_own [T, 1, len, H]), then run ONE decode step over the whole batch in which the rows `rows` get the
    NumPy-drawn inputs xd_rows [T, len(rows), H].  Returns (cache, output [B, H], tap [L, 2, T, B, H])."""
    import torch
    B, ps, T, H = len(lens), wl.page_size, wl.T, wl.hidden
    pages = int(sum(-(-(int(n) + 1) // ps) for n in lens))
    cache = model.new_cache(pages, ps, kv_dtype="e4m3" if kv8 else "model")
    g = torch.Generator(device=model.device).manual_seed(seed)
    order = np.argsort(-np.asarray(lens), kind="stable")
    i = 0
    while i < B:
        n = int(lens[order[i]])
        j = i
        while j < B and int(lens[order[j]]) == n and (j == i or (j - i + 1) * n <= sub_tokens):
            j += 1
        ids = [int(s) for s in order[i:j]]
        x = torch.randn((T, len(ids), n, H), generator=g, device=model.device, dtype=torch.float32).to(torch.bfloat16)
        if own in ids:
            x[:, ids.index(own)] = Hp.to_dev(model, x_own[:, 0])
        model.prefill(cache, x, ids)
        i = j
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    xd = torch.randn((T, B, H), generator=g, device=model.device, dtype=torch.float32).to(torch.bfloat16)
    xd[:, rows] = Hp.to_dev(model, xd_rows)
    tap = model.set_tap(-1, B)
    got = model.decode_step(cache, xd.contiguous(), list(range(B)))
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    model.set_tap(None)
    for s in range(B):
        assert cache.length(s) == int(lens[s]) + 1
    return cache, got, tap


def _decode_against_oracle(model, wl, ws, lens, own, injected, seed, tag, sub_tokens=16384, kv8=False):
    """kv8: the cache holds E4M3 codes on both sides.  The device quantises the K and V its bf16 GEMM made, the
    oracle its exact ones, so cached values may sit one code step apart: the mean bound comes from the floor
    measured with that format, the cached values are held to one code step, a layer delta to 6e-2."""
    import torch
    T, L, ps = wl.T, wl.L, wl.page_size
    mean_tol = Hp.mean_bound(wl, kv8=kv8)
    rows = [own, injected]
    x_own = I.prefill_inputs(wl, batch=1, seq=int(lens[own]), salt=200)
    xd_rows = I.decode_inputs(wl, batch=2, step=0)
    cache, got, tap = _fill_and_decode(model, wl, lens, own, x_own, rows, xd_rows, seed, sub_tokens, kv8)
    cfg = Hp.oracle_cfg(wl)
    ocache = O.PagedKVCache(cfg, sum(-(-(int(lens[r]) + 1) // ps) for r in rows), ps, kv_format="e4m3" if kv8 else "model")
    O.pt_prefill(cfg, Hp.Prefetch(ws, T, L), x_own, ocache, [0])            # the oracle's own cache for `own`
    # the K/V the device cached for `own` against the oracle's: every track and layer, all whole pages (the tail
    # page has unwritten slots), accumulated track by track
    n_own = int(lens[own])
    full = n_own // ps
    pages = torch.tensor(cache.block_table(own)[:full], device=cache.pool.device)
    opages = np.asarray(ocache.block_table[0][:full])
    dmax = dsum = rmax = rsum = 0.0
    for t in range(T):
        want = ocache.pool[t][:, opages]
        have, sc = _seq_kv(cache, wl, t, pages)
        d = np.abs(have - want)
        if kv8:      # never further apart than the largest code step (32 units of the larger of the two scales)
            assert np.all(d <= 32.0 * np.maximum(sc, ocache.scale[t][:, opages])[..., None] * (1 + 1e-6))
        dmax, dsum = max(dmax, float(d.max())), dsum + float(d.sum())
        rmax, rsum = max(rmax, float(np.abs(want).max())), rsum + float(np.abs(want).sum())
        del d, want, have
    mx, mean = dmax / rmax, dsum / rsum
    # bf16 cache: a cached value carries its own bf16 rounding on top of its projection's operand rounding, so the
    # mean bound is doubled; E4M3 cache: one code step of a value near the top of its binade is 32 / 224 of it
    kv_mx, kv_mean = (32.0 / 224.0, 1e-2) if kv8 else (2e-2, 2 * mean_tol)
    Hp.record(f"{tag}: cached K/V of the own-cache sequence ({full * ps} tokens, all tracks and layers)", mx, mean, kv_mx, kv_mean)
    assert mx <= kv_mx and mean <= kv_mean, f"cached K/V: max-rel {mx:.3e}, mean-rel {mean:.3e}"
    _inject(cache, wl, injected, int(lens[injected]), ocache, 1)
    taps = {}
    ref = O.pt_decode_step(cfg, Hp.Prefetch(ws, T, L), xd_rows, ocache, [0, 1], taps)
    out = got[rows].cpu().numpy()
    for i, (r, kind) in enumerate(zip(rows, ("own cache", "device cache"))):
        Hp.assert_close(out[i], ref[i], wl.dtype, f"{tag}: decode output of sequence {r}", mean_tol=mean_tol,
                        log=f"{tag}: decode output, sequence {r} (KV {int(lens[r])}, {kind})")
    tp = tap[:, :, :, rows].cpu().numpy()
    _check_taps(wl, tp, taps, 2, 1, mean_tol, delta_tol=6e-2 if kv8 else None)     # every layer's stream and both deltas
    for l in _tap_layers(wl) + [L - 1]:
        mx, mean = Hp.rel_errs(tp[l, 1], taps["h"][l].reshape(T, 2, wl.hidden))
        Hp.record(f"{tag}: layer {l} stream after the layer (both sequences)", mx, mean, 2e-2, mean_tol)
    cache.close()
    del cache, tap, pages
    torch.cuda.empty_cache()


@pytest.mark.parametrize("kv8", [False, True])
def test_decode_against_oracle_machinery_on_a_small_model(kv8):
    """The same own-cache / device-cache comparison on a model the oracle runs in a second."""
    wl = I.Workload("small-decode", T=3, L=6, D=3, hidden=256, heads=2 if kv8 else 4, kv_heads=1 if kv8 else 2, ffn=352,
                    dtype="bf16", mode="decode", batch=5, seq=0, ragged=(40, 200))
    ws = I.WeightSource(wl)
    model = Hp.make_model(wl, ws, max_pos=256)
    lens = I.kv_lengths(wl)
    _decode_against_oracle(model, wl, ws, lens, own=int(np.argmin(lens)), injected=int(np.argmax(lens)), seed=5,
                           tag="small ragged decode" + (" (e4m3 cache)" if kv8 else ""), sub_tokens=256, kv8=kv8)
    model.close()


def test_decode_full_size_matches_oracle_cfg2(mid_model):
    wl3, ws, model = mid_model
    wl = I.WORKLOADS["cfg2"]
    if _free_gib() < 133:
        pytest.skip(f"needs about 133 GiB of free device memory, {_free_gib():.0f} GiB are free")
    _decode_against_oracle(model, wl, ws, I.kv_lengths(wl), own=37, injected=3, seed=7, tag="cfg2 decode batch 64 at KV 2048")


@pytest.fixture(scope="module")
def wide_model():
    """The T=4, L=48 GQA model of the ragged decode workload with its seeded weights."""
    import torch
    torch.cuda.empty_cache()
    wl = I.WORKLOADS["cfg4"]
    ws = I.WeightSource(wl)
    m = Hp.make_model(wl, Hp.Prefetch(ws, wl.T, wl.L), max_pos=int(I.kv_lengths(wl).max()) + 16)
    yield wl, ws, m
    m.close()


def _largest_batch(wl, lens_all, bytes_per_element, reserve_gib):
    """The largest prefix (a multiple of 16) of the workload's sequences whose pages fit the free device memory."""
    import torch
    page_bytes = wl.T * wl.L * 2 * wl.kv_heads * wl.page_size * (wl.head_dim * bytes_per_element + (4 if bytes_per_element == 1 else 0))
    pages_of = (lens_all.astype(np.int64) + 1 + wl.page_size - 1) // wl.page_size
    budget = torch.cuda.mem_get_info()[0] - (reserve_gib << 30)
    B = wl.batch
    while B > 16 and int(pages_of[:B].sum()) * page_bytes > budget:
        B -= 16
    return B if int(pages_of[:B].sum()) * page_bytes <= budget else 0


def test_decode_full_size_matches_oracle_cfg4_ragged_gqa(wide_model):
    """The wide GQA model at its full width and depth with the seeded weights and the seeded ragged lengths; the
    batch is the largest prefix of the 256 sequences whose pages fit the device, as in the benchmark.  The
    oracle's own-cache sequence is the shortest of the batch, the device-cache one the longest."""
    import torch
    wl, ws, model = wide_model
    torch.cuda.empty_cache()
    lens_all = I.kv_lengths(wl)
    B = _largest_batch(wl, lens_all, 2, 14)
    if not B:
        pytest.skip("not enough free device memory for 16 sequences")
    lens = lens_all[:B]
    _decode_against_oracle(model, wl, ws, lens, own=int(np.argmin(lens)), injected=int(np.argmax(lens)), seed=9,
                           tag=f"cfg4 ragged GQA decode batch {B}", sub_tokens=8192)


def test_decode_full_size_matches_oracle_cfg4_whole_batch_e4m3_cache(wide_model):
    """The same workload with the cache in the E4M3 format: all 256 sequences fit."""
    import torch
    wl, ws, model = wide_model
    torch.cuda.empty_cache()
    lens_all = I.kv_lengths(wl)
    B = _largest_batch(wl, lens_all, 1, 14)
    if B < wl.batch:
        pytest.skip(f"only {B} of {wl.batch} sequences fit the free device memory")
    _decode_against_oracle(model, wl, ws, lens_all, own=int(np.argmin(lens_all)), injected=int(np.argmax(lens_all)), seed=9,
                           tag=f"cfg4 ragged GQA decode batch {B}, e4m3 cache", sub_tokens=8192, kv8=True)


def test_wide_gqa_architecture_at_reduced_depth_matches_oracle():
    """The wide model's layer (hidden 2048, 16 query / 4 KV heads of 128, SwiGLU 5632, T=4) with one
    track block of depth 2 and a small ragged batch: prefill, then two decode steps, all against the oracle."""
    from tests.test_gpu_parity import run_case
    base = I.WORKLOADS["cfg4"]
    wl = I.Workload("cfg4-shallow", T=base.T, L=2, D=2, hidden=base.hidden, heads=base.heads, kv_heads=base.kv_heads,
                    ffn=base.ffn, dtype="bf16", mode="decode", batch=3, seq=0, ragged=base.ragged)
    run_case(wl, B=3, S=150, chunks=[130, 20], decode_steps=2, shuffle=True, mean_tol=Hp.mean_bound(wl))
