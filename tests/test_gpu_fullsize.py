"""Parity at the full sizes of the decode and prefill workloads, in the launch configuration the
benchmark times.

The CPU oracle cannot run these workloads whole, so each is tied to it through outputs the oracle
can compute one by one, or through properties that hold at any size:

  * prefill (T=8, L=32, 8 x 4096 tokens): causal attention makes the outputs of the first n tokens
    of a batch row depend on those n tokens only, so the oracle runs n tokens of sampled rows alone
    and its result is compared with the same positions of the full-size launch (final output, the
    residual stream of the last layer, cached K/V of the sampled positions);
  * decode (batch 64 at KV 2048; ragged GQA batch at the wide model): a decode step at position n
    equals row n of a prefill (Algorithm 1 does not know how tokens arrive), so every sequence's
    decode output is compared with the last row of a full-size prefill of the same tokens, which
    goes through different kernels (flash prefill against split-KV decode, large-M against
    small-M GEMM tiles).  The prefill side is what the first item pins to the oracle.
"""
import numpy as np
import pytest

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I
from tests import helpers as Hp

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
    m = Hp.make_model(wl, ws, max_pos=4096)
    yield wl, ws, m
    m.close()


def test_prefill_full_size_sampled_prefixes_match_oracle(mid_model):
    import torch
    wl, ws, model = mid_model
    B, S, ps = wl.batch, wl.seq, wl.page_size
    if _free_gib() < 60:
        pytest.skip("needs about 60 GiB of free device memory")
    pages = B * (S // ps)
    order = I.free_list_permutation(pages, seed=3)
    cache = model.new_cache(pages, ps, order)
    g = torch.Generator(device="cpu").manual_seed(1234)
    # inputs N(0, 1) rounded to bf16; the sampled rows are drawn with the NumPy recipe so the oracle sees the same values
    rows, n = [5, 2], 77                                   # sampled batch rows and the prefix length the oracle runs
    x = torch.randn((wl.T, B, S, wl.hidden), generator=g, dtype=torch.float32).to(torch.bfloat16)
    xs = I.prefill_inputs(wl, batch=len(rows), seq=n, salt=100)              # [T, 2, n, H], bf16-rounded NumPy draws
    for i, b in enumerate(rows):
        x[:, b, :n] = torch.from_numpy(xs[:, i]).to(torch.bfloat16)
    tap = model.set_tap(wl.L - 1, B * S)                   # residual stream of the last layer only
    seq_ids = [11 + 2 * b for b in range(B)]
    got = model.prefill(cache, x.to(model.device), seq_ids)
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    model.set_tap(None)
    cfg = Hp.oracle_cfg(wl)
    ocache = O.PagedKVCache(cfg, len(rows) * (-(-n // ps)), ps)
    taps = {}
    ref = O.pt_prefill(cfg, ws, xs, ocache, list(range(len(rows))), taps)    # [2, n, H]; weights generated once
    for i, b in enumerate(rows):
        Hp.assert_close(got[b, :n].cpu().numpy(), ref[i], wl.dtype, f"row {b}: final output of the first {n} tokens",
                        mean_tol=Hp.DEEP_MEAN_TOL)
        # last layer, after its attention residual add, every track (the stream before the final sum)
        h_attn = np.stack([taps["h"][wl.L - 2][t][i] + taps["attn_delta"][(t, wl.L - 1)][i] for t in range(wl.T)])
        got_attn = tap[0, 0, :, b * S:b * S + n].cpu().numpy()
        Hp.assert_close(got_attn, h_attn, wl.dtype, f"row {b}: last layer's stream after attention", mean_tol=Hp.DEEP_MEAN_TOL)
        # cached K/V of sampled positions in the first and last layer, through the library's own slot arithmetic
        pool = cache.pool
        for l in (0, wl.L - 1):
            for t in (0, wl.T - 1):
                for pos in (0, n // 2, n - 1):
                    for kv in (0, 1):
                        off = cache.slot(t, l, seq_ids[b], pos, kv, 3)
                        dev = pool[off:off + wl.head_dim].float().cpu().numpy()
                        page, slot = ocache.locate(i, pos)
                        want = ocache.pool[t, l, page, kv, 3, slot]
                        d = np.abs(dev - want)
                        assert d.max() <= 2e-2 * np.abs(want).max() + 1e-6, f"row {b} layer {l} track {t} pos {pos} kv {kv}"
    cache.close()
    del cache, x, tap
    torch.cuda.empty_cache()


def _decode_equals_prefill_row(model, wl, lens, seed, sub_tokens=16384):
    """Prefill len+1 tokens per sequence (in sub-batches), keep each sequence's last output row, drop
    the last token from every sequence, replay it as a decode step over the whole batch."""
    import torch
    B, ps, T, H = len(lens), wl.page_size, wl.T, wl.hidden
    pages = int(sum(-(-(int(n) + 1) // ps) for n in lens))
    cache = model.new_cache(pages, ps)
    g = torch.Generator(device=model.device).manual_seed(seed)
    last_x = torch.empty((T, B, H), dtype=torch.bfloat16, device=model.device)
    last_out = torch.empty((B, H), dtype=torch.float32, device=model.device)
    order = np.argsort(-np.asarray(lens), kind="stable")
    i = 0
    while i < B:
        n = int(lens[order[i]]) + 1
        j = i
        while j < B and int(lens[order[j]]) + 1 == n and (j == i or (j - i + 1) * n <= sub_tokens):
            j += 1
        ids = [int(s) for s in order[i:j]]
        x = torch.randn((T, len(ids), n, H), generator=g, device=model.device, dtype=torch.float32).to(torch.bfloat16)
        out = model.prefill(cache, x, ids)
        last_x[:, ids] = x[:, :, n - 1]
        last_out[ids] = out[:, n - 1]
        i = j
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    for s in range(B):
        cache.truncate(s, int(lens[s]))
    got = model.decode_step(cache, last_x.contiguous(), list(range(B)))
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    for s in range(B):
        assert cache.length(s) == int(lens[s]) + 1
    a, b = got.cpu().numpy().astype(np.float64), last_out.cpu().numpy().astype(np.float64)
    assert np.all(np.isfinite(a))
    # two bf16 computations of the same value (different tilings and summation orders): each is
    # within the bf16 bounds of the exact result, so they are within twice those bounds of each other
    mx, mean = Hp.rel_errs(a, b)
    assert mx <= 4e-2 and mean <= 2 * Hp.DEEP_MEAN_TOL, f"decode vs prefill row: max-rel {mx:.3e}, mean-rel {mean:.3e}"
    cache.close()
    del cache
    torch.cuda.empty_cache()


def test_decode_full_size_equals_prefill_row_cfg2(mid_model):
    wl3, ws, model = mid_model
    wl = I.WORKLOADS["cfg2"]
    if _free_gib() < 133:
        pytest.skip(f"needs about 133 GiB of free device memory, {_free_gib():.0f} GiB are free")
    _decode_equals_prefill_row(model, wl, I.kv_lengths(wl), seed=7)


def test_decode_full_size_equals_prefill_row_cfg4_ragged_gqa():
    """The wide GQA model at its full width and depth with the seeded ragged lengths; the batch is the
    largest prefix of the 256 sequences whose pages fit the device, as in the benchmark."""
    import torch
    from paper_2602_07306_b200 import pt
    wl = I.WORKLOADS["cfg4"]
    lens_all = I.kv_lengths(wl)
    model = pt.Model(T=wl.T, D=wl.D, L=wl.L, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads, ffn=wl.ffn,
                     dtype="bf16", max_pos=int(lens_all.max()) + 16)
    model.init_random(seed=0)
    page_bytes = wl.T * wl.L * 2 * wl.kv_heads * wl.page_size * wl.head_dim * 2
    pages_of = (lens_all.astype(np.int64) + 1 + wl.page_size - 1) // wl.page_size
    budget = torch.cuda.mem_get_info()[0] - (12 << 30)
    B = wl.batch
    while B > 16 and int(pages_of[:B].sum()) * page_bytes > budget:
        B -= 16
    if int(pages_of[:B].sum()) * page_bytes > budget:
        pytest.skip("not enough free device memory for 16 sequences")
    _decode_equals_prefill_row(model, wl, lens_all[:B], seed=9, sub_tokens=8192)
    model.close()


def test_wide_gqa_architecture_at_reduced_depth_matches_oracle():
    """The wide model's layer (hidden 2048, 16 query / 4 KV heads of 128, SwiGLU 5632, T=4) with one
    track block of depth 2 and a small ragged batch: prefill, then two decode steps, all against the oracle."""
    from tests.test_gpu_parity import run_case
    base = I.WORKLOADS["cfg4"]
    wl = I.Workload("cfg4-shallow", T=base.T, L=2, D=2, hidden=base.hidden, heads=base.heads, kv_heads=base.kv_heads,
                    ffn=base.ffn, dtype="bf16", mode="decode", batch=3, seq=0, ragged=base.ragged)
    run_case(wl, B=3, S=150, chunks=[130, 20], decode_steps=2, shuffle=True, mean_tol=Hp.WIDE_MEAN_TOL)
