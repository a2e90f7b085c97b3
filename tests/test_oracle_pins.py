"""Pins for the CPU oracle: every check compares it with something other than itself
(values the paper prints, closed forms, library routines, an independently written
single-track decoder, invariants of Algorithm 1, brute force)."""
import itertools
import os

import numpy as np
import pytest
import torch

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rows(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return [ln.split() for ln in f if ln.strip() and not ln.startswith("#")]


def tiny(T=2, L=4, D=2, H=32, nq=4, nkv=2, F=48, dtype="f32", **kw):
    wl = I.Workload("tiny", T=T, L=L, D=D, hidden=H, heads=nq, kv_heads=nkv, ffn=F,
                    dtype=dtype, mode="prefill", batch=2, seq=12, seed=3)
    cfg = O.PTConfig(T=T, D=D, L=L, hidden=H, heads=nq, kv_heads=nkv, ffn=F, **kw)
    return wl, cfg


def run_prefill(wl, cfg, ws, x, seq_ids=None, pages=64, free_order=None, taps=None, cache=None):
    cache = cache or O.PagedKVCache(cfg, pages, wl.page_size, free_order)
    seq_ids = list(range(x.shape[1])) if seq_ids is None else seq_ids
    return O.pt_prefill(cfg, ws, x, cache, seq_ids, taps), cache


# ---------------------------------------------------------------- values the paper prints

def test_sync_point_counts_match_paper():
    for L, D, tp, pt, frac in _rows("sync_points.txt"):
        L, D = int(L), int(D)
        assert O.sync_points_tp(L) == int(tp)
        assert O.sync_points_pt(L, D) == int(pt)
        assert O.sync_fraction_removed(L, D) == pytest.approx(float(frac), abs=0)
    # "16x" at D = 8
    assert O.sync_points_tp(48) / O.sync_points_pt(48, 8) == 16


def test_table1_head_partition():
    for _, layers, tq, pq, tkv, pkv, tracks in _rows("table1_heads.txt"):
        assert int(pq) * int(tracks) == int(tq) and int(pkv) * int(tracks) == int(tkv)
        # a per-track config with those heads is accepted and groups q heads evenly
        cfg = O.PTConfig(T=int(tracks), D=8, L=int(layers) // 8 * 8, hidden=int(pq) * 16,
                         heads=int(pq), kv_heads=int(pkv), ffn=32)
        assert cfg.group == int(pq) // int(pkv)


def test_oracle_counts_syncs_during_forward():
    wl, cfg = tiny(L=6, D=3)
    taps = {}
    run_prefill(wl, cfg, I.WeightSource(wl), I.prefill_inputs(wl), taps=taps)
    assert taps["syncs"] == 2
    with pytest.raises(ValueError):
        O.PTConfig(T=2, D=4, L=6, hidden=32, heads=4, kv_heads=2, ffn=48)


# ---------------------------------------------------------------- closed forms

@pytest.mark.parametrize("op", ["sum", "mean"])
def test_zero_output_projections_give_closed_form(op):
    """Wo = Wd = 0 makes every layer the identity, so only the sync schedule acts:
    out = T^(L/D - 1) * sum_t x_t for SUM, mean_t x_t for MEAN."""
    wl, cfg = tiny(T=3, L=6, D=2, sync_op=op)
    ws = I.WeightSource(wl, zero=("wo", "wd"))
    x = I.prefill_inputs(wl)
    out, _ = run_prefill(wl, cfg, ws, x)
    xs = x.astype(np.float64)
    want = 3 ** (6 // 2 - 1) * xs.sum(0) if op == "sum" else xs.mean(0)
    np.testing.assert_allclose(out, want, rtol=1e-13)
    xsh = I.prefill_inputs(wl, shared=True)
    out2, _ = run_prefill(wl, cfg, ws, xsh)
    want2 = 3 ** (6 // 2) * xsh[0].astype(np.float64) if op == "sum" else xsh[0]
    np.testing.assert_allclose(out2, want2, rtol=1e-13)


def test_single_token_layer_by_hand():
    """S = 1: softmax over one key is 1, attention returns v of the mapped KV head, RoPE at
    position 0 is the identity; the layer is then plain algebra, written out with loops."""
    wl, cfg = tiny(T=1, L=1, D=1, H=8, nq=4, nkv=2, F=6)
    ws = I.WeightSource(wl, gain_jitter=0.3)
    w = {k: v.astype(np.float64) for k, v in ws.get(0, 0).items()}
    x = I.prefill_inputs(wl, batch=1, seq=1)
    out, _ = run_prefill(wl, cfg, ws, x)
    h = x[0, 0, 0].astype(np.float64)
    H, dh, G = 8, 2, 2
    a = [h[i] / np.sqrt(sum(h[j] ** 2 for j in range(H)) / H + 1e-6) * w["g1"][i] for i in range(H)]
    v = [sum(w["wv"][r, i] * a[i] for i in range(H)) for r in range(2 * dh)]
    o = []
    for head in range(4):
        kvh = head // G
        o += [v[kvh * dh + d] for d in range(dh)]
    h1 = [h[r] + sum(w["wo"][r, i] * o[i] for i in range(H)) for r in range(H)]
    c = [h1[i] / np.sqrt(sum(z * z for z in h1) / H + 1e-6) * w["g2"][i] for i in range(H)]
    z = []
    for f in range(6):
        g = sum(w["wg"][f, i] * c[i] for i in range(H))
        u = sum(w["wu"][f, i] * c[i] for i in range(H))
        z.append(g / (1 + np.exp(-g)) * u)
    want = [h1[r] + sum(w["wd"][r, f] * z[f] for f in range(6)) for r in range(H)]
    np.testing.assert_allclose(out[0, 0], want, rtol=1e-12)


# ---------------------------------------------------------------- library routines

def test_pieces_against_torch_float64():
    rng = np.random.default_rng(0)
    h = rng.standard_normal((5, 7, 16))
    g = rng.standard_normal(16)
    want = torch.nn.functional.rms_norm(torch.from_numpy(h), (16,), torch.from_numpy(g), eps=1e-6)
    np.testing.assert_allclose(O.rmsnorm(h, g, 1e-6), want.numpy(), rtol=1e-13)
    z = rng.standard_normal(100) * 4
    np.testing.assert_allclose(O.silu(z), torch.nn.functional.silu(torch.from_numpy(z)).numpy(), rtol=1e-13)
    # causal attention, GQA by explicit head duplication on the torch side
    S, nq, nkv, dh = 9, 6, 2, 8
    q, k, v = rng.standard_normal((S, nq, dh)), rng.standard_normal((S, nkv, dh)), rng.standard_normal((S, nkv, dh))
    kk = np.repeat(k, nq // nkv, axis=1)
    vv = np.repeat(v, nq // nkv, axis=1)
    tq, tk, tv = (torch.from_numpy(a).permute(1, 0, 2)[None] for a in (q, kk, vv))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0].permute(1, 0, 2)
    np.testing.assert_allclose(O.attention(q, k, v, np.arange(S)), want.numpy(), rtol=1e-12, atol=1e-14)
    # a query at position p with more keys cached than it may see (decode-style mask)
    got = O.attention(q[4:5], k, v, np.array([4]))
    np.testing.assert_allclose(got[0], want.numpy()[4], rtol=1e-12, atol=1e-14)


def test_rope_properties():
    rng = np.random.default_rng(1)
    dh = 16
    u = rng.standard_normal((6, 3, dh))
    pos = np.array([0, 1, 5, 17, 100, 4095])
    r = O.rope(u, pos, 10000.0)
    np.testing.assert_array_equal(r[0], u[0])                               # position 0: identity
    np.testing.assert_allclose(np.linalg.norm(r, axis=-1), np.linalg.norm(u, axis=-1), rtol=1e-13)
    # <R_m q, R_n k> depends on m - n only
    q, k = rng.standard_normal((1, 1, dh)), rng.standard_normal((1, 1, dh))
    def dot(m, n):
        return float(np.sum(O.rope(q, np.array([m]), 1e4) * O.rope(k, np.array([n]), 1e4)))
    assert dot(7, 3) == pytest.approx(dot(104, 100), rel=1e-11)
    assert dot(7, 3) != pytest.approx(dot(7, 4), rel=1e-6)
    # pair j is rotated by pos * base^(-2j/dh): check one pair against a 2x2 rotation
    j, p = 3, 17
    ang = p * 10000.0 ** (-2 * j / dh)
    R = np.array([[np.cos(ang), -np.sin(ang)], [np.sin(ang), np.cos(ang)]])
    np.testing.assert_allclose(r[3, 1, [j, j + dh // 2]], R @ u[3, 1, [j, j + dh // 2]], rtol=1e-12)
    # the lowest pair turns by exactly pos radians
    ang0 = np.arctan2(r[1, 0, dh // 2], r[1, 0, 0]) - np.arctan2(u[1, 0, dh // 2], u[1, 0, 0])
    assert np.isclose((ang0 - 1.0 + np.pi) % (2 * np.pi) - np.pi, 0, atol=1e-12)


# ---------------------------------------------------------------- independent single-track decoder

def _torch_decoder(wl, ws, x):
    """A standard pre-norm decoder written with torch float64 library ops only (T = 1)."""
    F = torch.nn.functional
    H, nq, nkv, dh = wl.hidden, wl.heads, wl.kv_heads, wl.head_dim
    h = torch.from_numpy(x[0].astype(np.float64))
    B, S, _ = h.shape
    inv = 1.0 / (wl.rope_base ** (torch.arange(0, dh, 2, dtype=torch.float64) / dh))
    ang = torch.arange(S, dtype=torch.float64)[:, None] * inv[None]
    cos, sin = torch.cat([ang.cos(), ang.cos()], -1), torch.cat([ang.sin(), ang.sin()], -1)
    def rot(u):                                      # u [B, heads, S, dh]
        u1, u2 = u[..., : dh // 2], u[..., dh // 2:]
        return u * cos + torch.cat([-u2, u1], -1) * sin
    for l in range(wl.L):
        w = {k: torch.from_numpy(v.astype(np.float64)) for k, v in ws.get(0, l).items()}
        a = F.rms_norm(h, (H,), w["g1"], eps=wl.rms_eps)
        q = F.linear(a, w["wq"]).view(B, S, nq, dh).transpose(1, 2)
        k = F.linear(a, w["wk"]).view(B, S, nkv, dh).transpose(1, 2)
        v = F.linear(a, w["wv"]).view(B, S, nkv, dh).transpose(1, 2)
        q, k = rot(q), rot(k)
        k, v = k.repeat_interleave(nq // nkv, 1), v.repeat_interleave(nq // nkv, 1)
        o = F.scaled_dot_product_attention(q, k, v, is_causal=True).transpose(1, 2).reshape(B, S, nq * dh)
        h = h + F.linear(o, w["wo"])
        c = F.rms_norm(h, (H,), w["g2"], eps=wl.rms_eps)
        h = h + F.linear(F.silu(F.linear(c, w["wg"])) * F.linear(c, w["wu"]), w["wd"])
    return h.numpy()


def test_single_track_equals_standard_decoder():
    wl, cfg = tiny(T=1, L=4, D=2, H=48, nq=6, nkv=2, F=80)
    ws = I.WeightSource(wl, std=0.2, gain_jitter=0.2)
    x = I.prefill_inputs(wl)
    out, _ = run_prefill(wl, cfg, ws, x)
    np.testing.assert_allclose(out, _torch_decoder(wl, ws, x), rtol=1e-10, atol=1e-12)


def test_gqa_special_cases():
    # duplicated KV heads under MHA == GQA with the un-duplicated weights
    wl_g, cfg_g = tiny(T=2, H=32, nq=4, nkv=2)
    wl_m, cfg_m = tiny(T=2, H=32, nq=4, nkv=4)
    ws_g = I.WeightSource(wl_g, std=0.2)

    class Dup:
        def get(self, t, l):
            w = dict(ws_g.get(t, l))
            dh = wl_g.head_dim
            for k in ("wk", "wv"):
                w[k] = np.repeat(w[k].reshape(2, dh, -1), 2, axis=0).reshape(4 * dh, -1)
            return w
    x = I.prefill_inputs(wl_g)
    out_g, _ = run_prefill(wl_g, cfg_g, ws_g, x)
    out_m, _ = run_prefill(wl_m, cfg_m, Dup(), x)
    np.testing.assert_allclose(out_g, out_m, rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- invariants of Algorithm 1

def test_tracks_independent_between_syncs_and_equal_after():
    wl, cfg = tiny(T=3, L=4, D=2)
    ws = I.WeightSource(wl, std=0.2)
    x = I.prefill_inputs(wl)
    t0, t1 = {}, {}
    run_prefill(wl, cfg, ws, x, taps=t0)
    x2 = x.copy()
    x2[1] += 0.5                                     # perturb track 1 only
    run_prefill(wl, cfg, ws, x2, taps=t1)
    for l in range(cfg.D - 1):                       # layers before the first sync
        np.testing.assert_array_equal(t0["h"][l][0], t1["h"][l][0])
        np.testing.assert_array_equal(t0["h"][l][2], t1["h"][l][2])
        assert np.abs(t0["h"][l][1] - t1["h"][l][1]).max() > 1e-3
    for l in (1, 3):                                 # after a sync every track holds the same h
        for t in range(1, 3):
            np.testing.assert_array_equal(t0["h"][l][0], t0["h"][l][t])
    assert np.abs(t0["h"][1][0] - t1["h"][1][0]).max() > 1e-3     # the sync does mix track 1 in
    # between the syncs tracks differ (their weights differ)
    assert np.abs(t0["h"][2][0] - t0["h"][2][1]).max() > 1e-3


def test_track_permutation_invariance():
    wl, cfg = tiny(T=3, L=4, D=2)
    ws = I.WeightSource(wl, std=0.2)
    perm = [2, 0, 1]

    class Perm:
        def get(self, t, l):
            return ws.get(perm[t], l)
    x = I.prefill_inputs(wl)
    a, _ = run_prefill(wl, cfg, ws, x)
    b, _ = run_prefill(wl, cfg, Perm(), x[perm])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)


def test_causal_prefix_invariance():
    wl, cfg = tiny()
    ws = I.WeightSource(wl, std=0.2)
    x = I.prefill_inputs(wl, seq=12)
    full, _ = run_prefill(wl, cfg, ws, x)
    x2 = x.copy()
    x2[:, :, 7:] = I.prefill_inputs(wl, seq=12, salt=9)[:, :, 7:]
    changed, _ = run_prefill(wl, cfg, ws, x2)
    short, _ = run_prefill(wl, cfg, ws, x[:, :, :7])
    np.testing.assert_allclose(changed[:, :7], full[:, :7], rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(short, full[:, :7], rtol=1e-12, atol=1e-13)
    assert np.abs(changed[:, 7:] - full[:, 7:]).max() > 1e-3


@pytest.mark.parametrize("shuffle", [False, True])
def test_decode_equals_prefill_row_and_chunked_prefill(shuffle):
    wl, cfg = tiny(T=2, L=4, D=2)
    ws = I.WeightSource(wl, std=0.2)
    S = 37                                            # crosses two page boundaries, last page partial
    x = I.prefill_inputs(wl, batch=2, seq=S)
    order = I.free_list_permutation(16, seed=5) if shuffle else None
    full, _ = run_prefill(wl, cfg, ws, x, pages=16, free_order=order)
    # prefill n tokens, then decode the rest one by one
    n = 30
    cache = O.PagedKVCache(cfg, 16, 16, order)
    first = O.pt_prefill(cfg, ws, x[:, :, :n], cache, [0, 1])
    np.testing.assert_allclose(first, full[:, :n], rtol=1e-12, atol=1e-13)
    for p in range(n, S):
        row = O.pt_decode_step(cfg, ws, x[:, :, p], cache, [0, 1])
        np.testing.assert_allclose(row, full[:, p], rtol=1e-12, atol=1e-13)
    assert cache.length == {0: S, 1: S}
    # chunked prefill 16 + 21 equals one prefill
    cache2 = O.PagedKVCache(cfg, 16, 16, order)
    O.pt_prefill(cfg, ws, x[:, :, :16], cache2, [0, 1])
    second = O.pt_prefill(cfg, ws, x[:, :, 16:], cache2, [0, 1])
    np.testing.assert_allclose(second, full[:, 16:], rtol=1e-12, atol=1e-13)


def test_batch_rows_independent():
    wl, cfg = tiny()
    ws = I.WeightSource(wl, std=0.2)
    x = I.prefill_inputs(wl, batch=3, seq=9)
    full, _ = run_prefill(wl, cfg, ws, x)
    one, _ = run_prefill(wl, cfg, ws, x[:, 1:2])
    np.testing.assert_allclose(one[0], full[1], rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- paged cache: brute force

def test_slot_offset_enumerates_pool_in_order():
    cfg = O.PTConfig(T=2, D=1, L=3, hidden=8, heads=4, kv_heads=2, ffn=8)
    P, ps = 5, 4
    expected = 0
    for t, l, page, kv, head, slot in itertools.product(range(2), range(3), range(P), range(2), range(2), range(ps)):
        assert O.kv_slot_offset(cfg, P, ps, t, l, page, kv, head, slot) == expected
        expected += cfg.head_dim
    cache = O.PagedKVCache(cfg, P, ps)
    assert cache.pool.size == expected
    # the pool array is indexed the same way: write through the API, find it at the flat offset
    cache.reserve(7, 6)
    k = np.arange(4.0).reshape(1, 2, 2) + 1
    cache.write(1, 2, 7, np.array([5]), k, -k)
    page, slot = cache.locate(7, 5)
    flat = cache.pool.reshape(-1)
    off = O.kv_slot_offset(cfg, P, ps, 1, 2, page, 0, 1, slot)
    np.testing.assert_array_equal(flat[off:off + 2], k[0, 1])
    off = O.kv_slot_offset(cfg, P, ps, 1, 2, page, 1, 0, slot)
    np.testing.assert_array_equal(flat[off:off + 2], -k[0, 0])
    assert np.count_nonzero(flat) == 8


def test_allocator_brute_force():
    cfg = O.PTConfig(T=1, D=1, L=1, hidden=4, heads=2, kv_heads=1, ffn=4)
    order = [3, 0, 4, 1, 2, 5]
    cache = O.PagedKVCache(cfg, 6, 4, order)
    cache.reserve(10, 5)        # 2 pages
    cache.reserve(11, 1)        # 1 page
    cache.reserve(10, 8)        # still 2 pages
    cache.reserve(10, 9)        # 3rd page
    assert cache.block_table == {10: [3, 0, 1], 11: [4]}
    assert cache.free == [2, 5]
    assert [cache.locate(10, p) for p in (0, 3, 4, 8)] == [(3, 0), (3, 3), (0, 0), (1, 0)]
    with pytest.raises(MemoryError):
        cache.reserve(11, 13)
    cache.release(10)
    assert cache.free == [2, 5, 3, 0, 1]
    with pytest.raises(ValueError):
        O.PagedKVCache(cfg, 4, 4, [0, 1, 1, 2])


def test_cache_holds_rotated_keys_and_plain_values():
    """What is cached: K after the rotary embedding, V as projected."""
    wl, cfg = tiny(T=1, L=1, D=1, H=16, nq=2, nkv=1, F=8)
    ws = I.WeightSource(wl, std=0.3)
    x = I.prefill_inputs(wl, batch=1, seq=5)
    _, cache = run_prefill(wl, cfg, ws, x)
    w = {k: v.astype(np.float64) for k, v in ws.get(0, 0).items()}
    h = x[0, 0].astype(np.float64)
    a = h / np.sqrt((h * h).mean(-1, keepdims=True) + 1e-6)
    k, v = cache.gather(0, 0, 0, 5)
    np.testing.assert_allclose(v[:, 0], a @ w["wv"].T, rtol=1e-12)
    kk = a @ w["wk"].T
    np.testing.assert_allclose(k[0, 0], kk[0], rtol=1e-12)                    # position 0 un-rotated
    np.testing.assert_allclose(np.linalg.norm(k[:, 0], axis=-1), np.linalg.norm(kk, axis=-1), rtol=1e-12)
    assert np.abs(k[3, 0] - kk[3]).max() > 1e-3


# ---------------------------------------------------------------- the input generators

def test_bf16_rounding_matches_torch():
    a = np.random.default_rng(0).standard_normal(10000).astype(np.float32) * 3
    a[:4] = [1.00390625, 1.01171875, -0.0, 65504.0]                          # ties and edge values
    want = torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    np.testing.assert_array_equal(I.round_to_bf16(a), want)
    np.testing.assert_array_equal(I.bits_to_f32(I.bf16_bits(want)), want)


def test_workload_recipe():
    wl = I.WORKLOADS["cfg4"]
    lens = I.kv_lengths(wl)
    assert lens.shape == (256,) and lens.min() >= 512 and lens.max() <= 4096
    np.testing.assert_array_equal(lens[:16], I.kv_lengths(wl, batch=16))
    assert I.WORKLOADS["cfg2"].params_per_track_layer() == 12845056
    assert I.WORKLOADS["cfg4"].params_per_track_layer() == 45088768
    w = I.WeightSource(I.WORKLOADS["cfg0"]).get(1, 2)
    assert w["wq"].shape == (128, 128) and w["wg"].shape == (512, 128) and w["wd"].shape == (128, 512)
    assert abs(float(w["wg"].std()) - 0.02) < 1e-3 and np.all(w["g1"] == 1)
    np.testing.assert_array_equal(w["wq"], I.WeightSource(I.WORKLOADS["cfg0"]).get(1, 2)["wq"])


# ----------------------------------------------------------------------------- ends of the model

def test_embedding_is_a_one_hot_product():
    rng = np.random.default_rng(0)
    table = rng.standard_normal((11, 6))
    tokens = np.array([[3, 0, 10], [7, 7, 1]])
    onehot = np.zeros(tokens.shape + (11,))
    for idx in np.ndindex(tokens.shape):
        onehot[idx + (tokens[idx],)] = 1.0
    assert np.array_equal(O.embed(table, tokens), onehot @ table)


def test_lm_head_against_torch_rms_norm_and_linear():
    import torch
    rng = np.random.default_rng(1)
    h, g, w = rng.standard_normal((5, 16)), 1 + 0.1 * rng.standard_normal(16), rng.standard_normal((9, 16))
    want = torch.nn.functional.linear(torch.nn.functional.rms_norm(torch.from_numpy(h), (16,), torch.from_numpy(g), 1e-6),
                                      torch.from_numpy(w)).numpy()
    assert np.allclose(O.lm_head(h, g, w, 1e-6), want, rtol=1e-12, atol=1e-12)


def test_greedy_takes_the_lowest_index_among_equal_maxima():
    assert O.greedy(np.array([[1.0, 5.0, 5.0, 2.0], [7.0, 7.0, 7.0, 7.0], [0.0, -1.0, 3.0, 3.0]])).tolist() == [1, 0, 2]


def test_generation_equals_teacher_forced_prefill():
    """Feeding the generated tokens back one at a time (decode steps) gives the same logits as one
    prefill over prompt + generated tokens: the cache and the positions line up at both ends."""
    wl = I.Workload("gen", T=2, L=4, D=2, hidden=32, heads=2, kv_heads=1, ffn=48, dtype="f32", mode="prefill", batch=2, seq=5)
    cfg = O.PTConfig(T=wl.T, D=wl.D, L=wl.L, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads, ffn=wl.ffn)
    ws = I.WeightSource(wl, std=0.3)
    rng = np.random.default_rng(2)
    V = 13
    table, gain, w_out = rng.standard_normal((V, wl.hidden)), 1 + 0.1 * rng.standard_normal(wl.hidden), rng.standard_normal((V, wl.hidden))
    prompt = rng.integers(0, V, (2, 5))
    cache = O.PagedKVCache(cfg, 8, 4)
    toks, logits = O.pt_generate(cfg, ws, table, gain, w_out, prompt, 4, cache, [0, 1])
    full = np.concatenate([prompt, toks[:, :3]], axis=1)                  # the last token is never fed back
    cache2 = O.PagedKVCache(cfg, 8, 4)
    x = O.embed(table, full)
    h = O.pt_prefill(cfg, ws, np.broadcast_to(x, (cfg.T,) + x.shape), cache2, [0, 1])
    want = O.lm_head(h[:, 4:], gain, w_out, cfg.rms_eps)                  # logits after positions 4..7
    assert np.allclose(logits, want, rtol=1e-9, atol=1e-9)
    assert np.array_equal(toks, O.greedy(want))
    assert cache.length[0] == cache.length[1] == 8


# ---------------------------------------------------------------- FP8 KV-cache format

def _e4m3_table():
    """Every finite non-negative E4M3 value, decoded from the bit fields (independent of e4m3_round)."""
    vals = []
    for code in range(0x7F):                          # 0x7F is NaN
        e, m = code >> 3, code & 7
        vals.append((m / 8.0) * 2.0 ** -6 if e == 0 else (1 + m / 8.0) * 2.0 ** (e - 7))
    return np.array(vals)


def test_e4m3_rounding_against_the_enumerated_format_and_torch():
    fmt = {k: float(v) for k, v in _rows("e4m3_format.txt")}
    table = _e4m3_table()
    assert len(table) == fmt["finite_codes_per_sign"] and table.max() == fmt["max_normal"] == O.E4M3_MAX
    assert table[1] == fmt["min_subnormal"] and table[8] == fmt["min_normal"]
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(20000) * s for s in (1e-3, 0.05, 1.0, 30.0, 300.0)])
    mids = (table[:-1] + table[1:]) / 2                # exact ties between neighbouring values
    x = np.concatenate([x, mids, -mids, table, -table, [0.0, 448.0, 449.0, 1e6, -1e6, 463.9, 464.1]])
    got = O.e4m3_round(x)
    # brute force: nearest table value, ties to the even code (= even mantissa bit), saturating
    a = np.minimum(np.abs(x), 448.0)
    d = np.abs(a[:, None] - table[None, :])
    best = d.min(axis=1)
    want = np.empty_like(a)
    for i in range(len(a)):
        cand = np.flatnonzero(d[i] == best[i])
        want[i] = table[[c for c in cand if c % 2 == 0][0]] if len(cand) > 1 else table[cand[0]]
    np.testing.assert_array_equal(got, np.copysign(want, x))
    assert np.all(np.isin(np.abs(got), table))
    # the library's conversion (round to nearest even; it does not saturate, so in-range values only)
    xin = x[np.abs(x) <= 448.0].astype(np.float32)
    lib = torch.from_numpy(xin).to(torch.float8_e4m3fn).to(torch.float32).numpy()
    np.testing.assert_array_equal(O.e4m3_round(xin.astype(np.float64)).astype(np.float32), lib)


def test_kv_scale_is_the_smallest_power_of_two_without_saturation():
    rng = np.random.default_rng(1)
    v = rng.standard_normal((200, 16)) * np.exp2(rng.integers(-20, 12, (200, 1)))
    v[0] = 0.0
    v[1] = 0.0; v[1, 3] = 448.0                        # exactly the largest code at scale 1
    v[2] = 0.0; v[2, 5] = -448.0000001
    s = O.kv_scale(v)
    assert s.shape == (200, 1) and s[0, 0] == 1.0 and s[1, 0] == 1.0 and s[2, 0] == 2.0
    assert O.kv_scale(np.array([[1e-40, 0.0]]))[0, 0] == 2.0 ** -100       # the floor of the scale
    for i in range(3, 200):
        amax = np.abs(v[i]).max()
        cands = [2.0 ** e for e in range(-60, 40) if amax / 2.0 ** e <= 448.0]
        assert s[i, 0] == min(cands)
        assert 224.0 < amax / s[i, 0] <= 448.0         # the largest element uses the top binade
    codes, s2 = O.kv_quantize(v)
    np.testing.assert_array_equal(s, s2)
    assert np.all(np.isin(np.abs(codes), _e4m3_table()))
    # round-trip bound: half a unit in the last place, relative 2^-4 for normal codes, absolute for subnormal ones
    back = codes * s
    err = np.abs(back - v)
    normal = np.abs(v) >= s * 2.0 ** -6
    assert np.all(err[normal] <= np.abs(v)[normal] * 2.0 ** -4 * (1 + 1e-12))
    assert np.all(err[~normal] <= (s * 2.0 ** -10 * np.ones_like(v))[~normal] * (1 + 1e-12))


def test_fp8_cache_quantises_what_it_stores_and_nothing_else():
    wl, cfg = tiny(T=2, L=2, D=1, H=32, nq=4, nkv=2)
    ws = I.WeightSource(wl, std=0.2)
    S = 21
    x = I.prefill_inputs(wl, batch=2, seq=S)
    exact, c0 = run_prefill(wl, cfg, ws, x, pages=8)
    c8 = O.PagedKVCache(cfg, 8, 16, kv_format="e4m3")
    got = O.pt_prefill(cfg, ws, x, c8, [0, 1])
    # layer 0 caches the same K/V in both runs (its inputs do not depend on any cache): the FP8 pool is the
    # quantisation of the exact pool, vector by vector, and its scales are the ones kv_scale gives
    for t in range(cfg.T):
        for seq in (0, 1):
            k, v = c0.gather(t, 0, seq, S)
            k8, v8 = c8.gather(t, 0, seq, S)
            for a, b in ((k, k8), (v, v8)):
                codes, s = O.kv_quantize(a)
                np.testing.assert_array_equal(b, codes * s)
    assert np.all(np.log2(c8.scale) == np.round(np.log2(c8.scale)))
    assert np.all(c0.scale == 1.0)
    # the output moves by the quantisation error of attention's inputs and by no more: a few percent of its scale
    rel = np.abs(got - exact).max() / np.abs(exact).max()
    assert 1e-4 < rel < 0.1
    # Algorithm 1's invariants survive: a decode step equals a prefill row, chunked prefill equals one prefill
    # (each vector is quantised on its own, so it does not matter in which call it was written)
    c8b = O.PagedKVCache(cfg, 8, 16, kv_format="e4m3")
    first = O.pt_prefill(cfg, ws, x[:, :, :10], c8b, [0, 1])
    np.testing.assert_allclose(first, got[:, :10], rtol=1e-12, atol=1e-13)
    rest = O.pt_prefill(cfg, ws, x[:, :, 10:S - 1], c8b, [0, 1])
    np.testing.assert_allclose(rest, got[:, 10:S - 1], rtol=1e-12, atol=1e-13)
    last = O.pt_decode_step(cfg, ws, x[:, :, S - 1], c8b, [0, 1])
    np.testing.assert_allclose(last, got[:, S - 1], rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- PT-MoE feed-forward

def test_moe_gates_by_hand_and_against_torch():
    # a hand-checked row: logits 1, 3, 3, 0 with top-2: experts 1 and 2 tie for the top, both chosen, half each
    g = O.moe_gates(np.array([[1.0, 3.0, 3.0, 0.0]]), 2)
    np.testing.assert_allclose(g, [[0.0, 0.5, 0.5, 0.0]])
    # a tie at the boundary of the choice: the lower index wins
    g = O.moe_gates(np.array([[2.0, 5.0, 2.0, 2.0]]), 2)
    e = np.exp(2.0 - 5.0)
    np.testing.assert_allclose(g, [[e / (1 + e), 1 / (1 + e), 0.0, 0.0]])
    rng = np.random.default_rng(0)
    logits = rng.standard_normal((50, 7, 6))
    for k in (1, 2, 6):
        got = O.moe_gates(logits, k)
        tl = torch.from_numpy(logits)
        vals, idx = torch.topk(tl, k, dim=-1)
        want = torch.zeros_like(tl).scatter(-1, idx, torch.softmax(vals, dim=-1)).numpy()
        np.testing.assert_allclose(got, want, rtol=1e-13, atol=1e-15)
        assert np.all((got > 0).sum(-1) == k) and np.allclose(got.sum(-1), 1.0)


def test_moe_ffn_special_cases():
    rng = np.random.default_rng(1)
    H, F, E, n = 16, 24, 4, 9
    c = rng.standard_normal((n, H))
    wr = rng.standard_normal((E, H))
    wg, wu, wd = rng.standard_normal((E, F, H)) * 0.3, rng.standard_normal((E, F, H)) * 0.3, rng.standard_normal((E, H, F)) * 0.3
    dense = lambda e: (O.silu(c @ wg[e].T) * (c @ wu[e].T)) @ wd[e].T
    # one expert: the plain feed-forward, whatever the router says
    np.testing.assert_allclose(O.moe_ffn(c, wr[:1], wg[:1], wu[:1], wd[:1], 1), dense(0), rtol=1e-13)
    # identical experts: the gates sum to one, so the mixture is that expert
    same = lambda a: np.repeat(a[:1], E, axis=0)
    np.testing.assert_allclose(O.moe_ffn(c, wr, same(wg), same(wu), same(wd), 2), dense(0), rtol=1e-12)
    # all experts chosen: a softmax mixture of every expert, written out
    p = torch.softmax(torch.from_numpy(c @ wr.T), dim=-1).numpy()
    np.testing.assert_allclose(O.moe_ffn(c, wr, wg, wu, wd, E), sum(p[:, e:e + 1] * dense(e) for e in range(E)), rtol=1e-12)
    # top-1 by brute force, token by token
    want = np.stack([dense(int(np.argmax(c[i] @ wr.T)))[i] for i in range(n)])
    np.testing.assert_allclose(O.moe_ffn(c, wr, wg, wu, wd, 1), want, rtol=1e-12)
    # renumbering the experts (router rows and expert weights together) changes nothing
    perm = np.array([2, 0, 3, 1])
    np.testing.assert_allclose(O.moe_ffn(c, wr[perm], wg[perm], wu[perm], wd[perm], 2), O.moe_ffn(c, wr, wg, wu, wd, 2), rtol=1e-12)


def test_moe_stack_reduces_to_the_dense_stack_with_one_expert_and_keeps_algorithm_1s_invariants():
    base = dict(T=2, L=4, D=2, hidden=32, heads=4, kv_heads=2, ffn=48, dtype="f32", mode="prefill", batch=2, seq=12, seed=3)
    wl1 = I.Workload("moe1", experts=1, top_k=1, **base)
    wl0 = I.Workload("dense", **base)
    ws1, ws0 = I.WeightSource(wl1, std=0.2), I.WeightSource(wl0, std=0.2)
    x = I.prefill_inputs(wl0)
    cfg0 = O.PTConfig(T=2, D=2, L=4, hidden=32, heads=4, kv_heads=2, ffn=48)
    cfg1 = O.PTConfig(T=2, D=2, L=4, hidden=32, heads=4, kv_heads=2, ffn=48, experts=1, top_k=1)

    class One:                                    # the dense weights, presented as one expert
        def get(self, t, l):
            w = dict(ws0.get(t, l))
            for k in ("wg", "wu", "wd"):
                w[k] = w[k][None]
            w["wr"] = ws1.get(t, l)["wr"]
            return w
    a = O.pt_prefill(cfg0, ws0, x, O.PagedKVCache(cfg0, 8, 16), [0, 1])
    b = O.pt_prefill(cfg1, One(), x, O.PagedKVCache(cfg1, 8, 16), [0, 1])
    np.testing.assert_allclose(a, b, rtol=1e-12, atol=1e-13)
    # four experts, top-2: decode equals a prefill row, and the sync count is still L / D
    wl4 = I.Workload("moe4", experts=4, top_k=2, **base)
    ws4 = I.WeightSource(wl4, std=0.2, router_std=0.5)
    cfg4 = O.PTConfig(T=2, D=2, L=4, hidden=32, heads=4, kv_heads=2, ffn=48, experts=4, top_k=2)
    taps = {}
    full = O.pt_prefill(cfg4, ws4, x, O.PagedKVCache(cfg4, 8, 16), [0, 1], taps)
    assert taps["syncs"] == 2 and taps["router_logits"][(1, 3)].shape == (2, 12, 4)
    cache = O.PagedKVCache(cfg4, 8, 16)
    O.pt_prefill(cfg4, ws4, x[:, :, :11], cache, [0, 1])
    last = O.pt_decode_step(cfg4, ws4, x[:, :, 11], cache, [0, 1])
    np.testing.assert_allclose(last, full[:, 11], rtol=1e-12, atol=1e-13)
    assert np.abs(full - a).max() > 1e-3          # and it is not the dense stack
    with pytest.raises(ValueError):
        O.PTConfig(T=2, D=2, L=4, hidden=32, heads=4, kv_heads=2, ffn=48, experts=4, top_k=5)
