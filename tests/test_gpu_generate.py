"""Ends of the model on the GPU against the oracle: embedding lookup (bit-exact gather), final RMSNorm +
LM head (logits within the bf16 bounds), the greedy choice (an integer decided by floating point: checked
bit-exactly against the device's own logits, and against the oracle's choice wherever the oracle's top-2
margin exceeds the logits' error), and the greedy generate loop."""
import numpy as np
import pytest

from oracle import pt_oracle as O
from paper_2602_07306_b200 import inputs as I
from tests import helpers as Hp

pytestmark = pytest.mark.gpu

V = 208                      # vocabulary (multiple of 16, N tail for 128-wide tiles)


def _setup(seed=0, T=2, L=4, D=2, H=256, nq=4, nkv=2, F=352):
    wl = I.Workload("gen", T=T, L=L, D=D, hidden=H, heads=nq, kv_heads=nkv, ffn=F, dtype="bf16", mode="prefill", batch=2, seq=8)
    ws = I.WeightSource(wl, std=0.05, gain_jitter=0.1)
    rng = np.random.default_rng(seed)
    table = I.round_to_bf16(rng.standard_normal((V, H), dtype=np.float32))
    head = I.round_to_bf16(rng.standard_normal((V, H), dtype=np.float32) * 0.3)
    head[17] = head[5]                                   # two identical rows: their logits tie exactly
    gain = (1 + 0.1 * rng.standard_normal(H)).astype(np.float32)
    model = Hp.make_model(wl, ws, max_pos=64)
    model.load_lm(table, head, gain)
    return wl, ws, model, table, head, gain


def test_embedding_is_an_exact_gather_and_bad_ids_are_reported():
    import torch
    wl, ws, model, table, head, gain = _setup()
    tok = np.array([[3, 0, V - 1], [7, 7, 100]], np.int32)
    x = model.embed(torch.from_numpy(tok).cuda())
    assert np.array_equal(x.float().cpu().numpy(), O.embed(table, tok).astype(np.float32))
    assert model.device_status() == (0, 0)
    bad = torch.tensor([1, V + 3], dtype=torch.int32).cuda()
    x = model.embed(bad)
    code, loc = model.device_status()
    assert code == 8 and np.array_equal(x[1].float().cpu().numpy(), table[0])
    model.close()


def test_lm_head_logits_and_greedy_choice():
    import torch
    wl, ws, model, table, head, gain = _setup(seed=1)
    rng = np.random.default_rng(5)
    h = (rng.standard_normal((37, wl.hidden)) * 3).astype(np.float32)
    h[4] = 0.0                                           # a zero row: every logit ties at 0 -> index 0
    logits, tok = model.lm_head(torch.from_numpy(h).cuda())
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    got = logits.cpu().numpy()
    ref = O.lm_head(h, gain, head, wl.rms_eps)
    Hp.assert_close(got, ref, "bf16", "logits")
    # the choice is exactly the lowest index of the device's own largest logit ...
    assert np.array_equal(tok.cpu().numpy(), np.argmax(got, axis=-1))
    assert tok[4].item() == 0
    tied = got[:, 17] == got[:, 5]
    assert tied.all() and not np.any(tok.cpu().numpy() == 17)            # identical rows tie bit for bit; 5 wins over 17
    # ... and the oracle's wherever its top-2 margin is larger than the logits' error
    err = np.abs(got - ref).max()
    srt = np.sort(ref, axis=-1)
    clear = (srt[:, -1] - srt[:, -2]) > 2 * err
    assert clear.sum() >= 20
    assert np.array_equal(tok.cpu().numpy()[clear], O.greedy(ref)[clear])
    model.close()


def test_greedy_generation_follows_the_oracle():
    import torch
    wl, ws, model, table, head, gain = _setup(seed=2)
    cfg = Hp.oracle_cfg(wl)
    rng = np.random.default_rng(9)
    B, S, n_new = 3, 21, 6
    prompt = rng.integers(0, V, (B, S)).astype(np.int32)
    pages = B * 3 + 1
    order = I.free_list_permutation(pages, seed=4)
    cache = model.new_cache(pages, 16, order)
    toks, logits = model.generate(cache, torch.from_numpy(prompt).cuda(), n_new, [4, 9, 2], want_logits=True)
    torch.cuda.synchronize()
    assert model.device_status() == (0, 0)
    toks, logits = toks.cpu().numpy(), logits.cpu().numpy()
    ocache = O.PagedKVCache(cfg, pages, 16, order)
    rtoks, rlogits = O.pt_generate(cfg, ws, table, gain, head, prompt, n_new, ocache, [4, 9, 2], round_x=I.round_to_bf16)
    for b in range(B):
        for i in range(n_new):
            # the device's choice is the argmax of the device's logits, always
            assert toks[b, i] == np.argmax(logits[b, i])
            mx, mean = Hp.rel_errs(logits[b, i], rlogits[b, i])
            assert mx <= 2e-2 and mean <= 4e-3, (b, i, mx, mean)
            if toks[b, i] != rtoks[b, i]:
                # two correct continuations: only allowed when the oracle's margin is inside the logits' error
                srt = np.sort(rlogits[b, i])
                assert srt[-1] - srt[-2] <= 2 * np.abs(logits[b, i] - rlogits[b, i]).max(), (b, i)
                break                                     # the sequences differ from here on
    for s in (4, 9, 2):
        assert cache.length(s) == S + n_new - 1 == ocache.length[s]
        assert cache.block_table(s) == ocache.block_table[s]
    model.close()
