"""PT-MoE (a mixture-of-experts feed-forward inside every track) on the GPU against the oracle.

The choice of experts is an integer decided by floating point: the device computes the router logits from the
bf16 operand of the feed-forward, the oracle in float64 (the logits then differ by some 1e-3 of their size), so
a token whose k-th and (k+1)-th logits nearly tie may choose differently on the two sides and then differs by a
whole expert.  Three cases deal with that:
  * one layer, 200 tokens, top 2 of 4: a layer's feed-forward touches only its own token, so the tokens whose
    decision has a margin above 1e-2 of the logits' size (nearly all) are compared row by row and the others are
    left out (and counted);
  * two layers, prefill and a decode step, seeded so that EVERY decision of the run has such a margin - the test
    checks that on the oracle's own logits before it compares anything;
  * all experts chosen (top_k = experts: no decision to take), a softmax mixture, at a larger size.
"""
import numpy as np
import pytest

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I
from tests import helpers as Hp
from tests.test_gpu_parity import _check_taps

pytestmark = pytest.mark.gpu


def _moe_wl(name, E, k, T=2, L=4, D=2, H=256, nq=4, nkv=2, F=176, seed=0):
    return I.Workload(name, T=T, L=L, D=D, hidden=H, heads=nq, kv_heads=nkv, ffn=F, dtype="bf16", mode="prefill",
                      batch=2, seq=24, seed=seed, experts=E, top_k=k)


def min_relative_margin(taps, top_k):
    """Smallest gap between the k-th and (k+1)-th largest router logit of any (track, layer, token), relative to
    the largest |logit| of that token."""
    worst = np.inf
    for lg in taps["router_logits"].values():
        srt = np.sort(lg, axis=-1)[..., ::-1]
        if top_k < srt.shape[-1]:
            gap = (srt[..., top_k - 1] - srt[..., top_k]) / np.abs(lg).max(axis=-1)
            worst = min(worst, float(gap.min()))
    return worst


MARGIN = 1e-2


def token_margins(taps, top_k):
    """Per token [B, S]: the smallest relative margin of its routing decisions over all tracks and layers."""
    worst = None
    for lg in taps["router_logits"].values():
        srt = np.sort(lg, axis=-1)[..., ::-1]
        gap = (srt[..., top_k - 1] - srt[..., top_k]) / np.abs(lg).max(axis=-1)
        worst = gap if worst is None else np.minimum(worst, gap)
    return worst


def run_moe(wl, ws, S, decode_steps, check_margin):
    import torch
    cfg = Hp.oracle_cfg(wl)
    B = wl.batch
    model = Hp.make_model(wl, ws, max_pos=64)
    pages = B * 4
    cache = model.new_cache(pages, 16)
    ocache = O.PagedKVCache(cfg, pages, 16)
    x = I.prefill_inputs(wl, batch=B, seq=S)
    for step in range(1 + decode_steps):
        taps = {}
        if step == 0:
            ref = O.pt_prefill(cfg, ws, x, ocache, [0, 1], taps)
            n = S
        else:
            xd = I.decode_inputs(wl, batch=B, step=step)
            ref = O.pt_decode_step(cfg, ws, xd, ocache, [0, 1], taps)
            n = 1
        if check_margin:
            margin = min_relative_margin(taps, wl.top_k)
            assert margin > MARGIN, f"seeded case has a near-tie in its routing (relative margin {margin:.2e}): pick another seed"
        tap = model.set_tap(-1, B * n)
        got = model.prefill(cache, Hp.to_dev(model, x), [0, 1]) if step == 0 else model.decode_step(cache, Hp.to_dev(model, xd), [0, 1])
        torch.cuda.synchronize()
        assert model.device_status() == (0, 0)
        Hp.assert_close(got.cpu().numpy(), ref, wl.dtype, f"{wl.name} step {step}", log=f"PT-MoE {wl.name}: {'prefill' if step == 0 else 'decode step %d' % step}")
        _check_taps(wl, tap.cpu().numpy(), taps, B, n)
    model.set_tap(None)
    model.close()


def test_moe_top2_of_4_one_layer_row_by_row():
    import torch
    wl = _moe_wl("top2of4-1layer", 4, 2, T=2, L=1, D=1, seed=1)
    ws = I.WeightSource(wl, gain_jitter=0.1, router_std=0.3)
    cfg = Hp.oracle_cfg(wl)
    B, S = 2, 100
    x = I.prefill_inputs(wl, batch=B, seq=S)
    taps = {}
    ref = O.pt_prefill(cfg, ws, x, O.PagedKVCache(cfg, 16, 16), [0, 1], taps)
    model = Hp.make_model(wl, ws, max_pos=128)
    got = model.prefill(model.new_cache(16, 16), Hp.to_dev(model, x), [0, 1]).cpu().numpy()
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    model.close()
    safe = token_margins(taps, wl.top_k) > MARGIN                  # [B, S]
    assert safe.mean() > 0.9, safe.mean()
    Hp.assert_close(got[safe], ref[safe], wl.dtype, "tokens with a clear routing decision",
                    log=f"PT-MoE top 2 of 4, one layer: {int(safe.sum())} of {safe.size} tokens with a routing margin above {MARGIN}")
    # the left-out tokens either routed the same way after all (and then agree) or took a neighbouring expert
    rest = np.abs(got[~safe] - ref[~safe]).max(axis=-1) / np.abs(ref).max() if (~safe).any() else np.zeros(0)
    print(f"left out: {int((~safe).sum())} tokens, of which {int((rest > 2e-2).sum())} differ by more than 2e-2 of the maximum")


def test_moe_top2_of_4_two_layers_prefill_and_decode():
    wl = _moe_wl("top2of4", 4, 2, L=2, D=1, seed=42)
    ws = I.WeightSource(wl, gain_jitter=0.1, router_std=0.3)
    run_moe(wl, ws, S=6, decode_steps=1, check_margin=True)


def test_moe_all_experts_is_a_softmax_mixture():
    wl = _moe_wl("all3", 3, 3, T=3, L=2, D=1, H=512, nq=8, nkv=8, F=208)
    ws = I.WeightSource(wl, gain_jitter=0.1, router_std=0.05)
    run_moe(wl, ws, S=24, decode_steps=1, check_margin=False)


def test_moe_with_one_expert_is_the_dense_model_bit_for_bit():
    import torch
    base = _moe_wl("dense", 0, 0)
    one = _moe_wl("one", 1, 1)
    ws0 = I.WeightSource(base, gain_jitter=0.1)

    class One:
        def get(self, t, l):
            w = dict(ws0.get(t, l))
            for k in ("wg", "wu", "wd"):
                w[k] = w[k][None]
            w["wr"] = np.ones((1, base.hidden), np.float32)
            return w
    x = I.prefill_inputs(base, batch=2, seq=24)
    outs = []
    for wl, ws in ((base, ws0), (one, One())):
        m = Hp.make_model(wl, ws, max_pos=64)
        cache = m.new_cache(8, 16)
        outs.append(m.prefill(cache, Hp.to_dev(m, x), [0, 1]).cpu().numpy())
        torch.cuda.synchronize()
        assert m.device_status() == (0, 0)
        m.close()
    np.testing.assert_array_equal(outs[0], outs[1])



# ---- the permuted-token path (prefill calls of 512 rows or more evaluate only the chosen experts)

def test_moe_sparse_all_experts_two_layers_with_a_sync():
    wl = _moe_wl("sparse-all3", 3, 3, T=2, L=2, D=2, H=256, nq=4, nkv=2, F=176)
    ws = I.WeightSource(wl, gain_jitter=0.1, router_std=0.05)
    import torch
    cfg = Hp.oracle_cfg(wl)
    B, S = 2, 300                                                  # 600 rows: the permuted path
    x = I.prefill_inputs(wl, batch=B, seq=S)
    taps = {}
    ref = O.pt_prefill(cfg, ws, x, O.PagedKVCache(cfg, 40, 16), [0, 1], taps)
    model = Hp.make_model(wl, ws, max_pos=320)
    tap = model.set_tap(-1, B * S)
    got = model.prefill(model.new_cache(40, 16), Hp.to_dev(model, x), [0, 1])
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    Hp.assert_close(got.cpu().numpy(), ref, wl.dtype, "permuted-token path, all experts", log="PT-MoE permuted tokens, all 3 experts, 600 rows: prefill")
    _check_taps(wl, tap.cpu().numpy(), taps, B, S)
    model.set_tap(None)
    model.close()


def test_moe_sparse_top2_of_4_row_by_row_and_against_the_dense_masked_path():
    import torch
    wl = _moe_wl("sparse-top2of4", 4, 2, T=2, L=1, D=1, seed=2)
    ws = I.WeightSource(wl, gain_jitter=0.1, router_std=0.3)
    cfg = Hp.oracle_cfg(wl)
    B, S = 2, 320
    x = I.prefill_inputs(wl, batch=B, seq=S)
    taps = {}
    ref = O.pt_prefill(cfg, ws, x, O.PagedKVCache(cfg, 40, 16), [0, 1], taps)
    model = Hp.make_model(wl, ws, max_pos=320)
    from paper_2602_07306_b200 import pt
    xd = Hp.to_dev(model, x)
    n0 = pt.lib().pt_launch_count()
    sparse = model.prefill(model.new_cache(40, 16), xd, [0, 1]).cpu().numpy()           # 640 rows at once
    # input prep + [QKV, attention, out-projection, router, plan, dispatch, gate/up, down, combine]
    assert pt.lib().pt_launch_count() - n0 == 1 + 9
    cache = model.new_cache(40, 16)                                                     # 2 x 160 rows per call: every expert for every token
    dense = np.concatenate([model.prefill(cache, xd[:, :, :160].contiguous(), [0, 1]).cpu().numpy(),
                            model.prefill(cache, xd[:, :, 160:].contiguous(), [0, 1]).cpu().numpy()], axis=1)
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    model.close()
    # one layer: both paths route from the same operand, so they take the same decisions; they differ in summation order only
    mx, mean = Hp.rel_errs(sparse, dense)
    Hp.record("PT-MoE top 2 of 4, one layer, 640 rows: permuted-token path against the dense-masked path", mx, mean, 1e-3, 1e-4)
    assert mx <= 1e-3 and mean <= 1e-4
    safe = token_margins(taps, wl.top_k) > MARGIN
    assert safe.mean() > 0.9
    Hp.assert_close(sparse[safe], ref[safe], wl.dtype, "tokens with a clear routing decision",
                    log=f"PT-MoE permuted tokens, top 2 of 4, one layer: {int(safe.sum())} of {safe.size} tokens with a routing margin above {MARGIN}")
