"""The E4M3 storage format of the KV cache on the GPU, against the oracle's.

  * the quantiser alone, bit for bit: scale and codes of crafted and random bf16 vectors (the decision which
    code a value gets is taken on the same bf16 inputs on both sides);
  * whole forwards with an E4M3 cache (chunked prefill with earlier context, decode steps over several key
    ranges, GQA groups of 1, 4 and 8, pages of 16 and 32 tokens, shuffled pages) against the oracle with the
    same cache format: final output and every layer's stream within 2e-2 of the maximum and within the mean
    bound derived from the measured floor (tests/bf16_floor.py with kv8: the device quantises the K and V its
    bf16 GEMM produced, the oracle its exact ones, so a value near a code boundary lands one code step away;
    that, not bf16 rounding, sets the floor); scales and cached values; page tables bit-exact.
"""
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
