"""Track parallelism across ranks (the paper's deployment: some tracks per GPU, one all-reduce per track
block).  One GPU is enough to check it end to end: a rank is a model that holds
part of the tracks plus an all-reduce hook, and two such ranks can share one GPU as long as their kernels
never wait for each other on the device - here the exchange is a host-side barrier between two threads."""
import threading

import numpy as np
import pytest

from paper_2602_07306_b200 import inputs as I
from tests import helpers as Hp

pytestmark = pytest.mark.gpu


class _Tracks:
    """Weights of tracks [lo, hi) of a larger stack, renumbered from 0."""
    def __init__(self, ws, lo):
        self.ws, self.lo = ws, lo

    def get(self, t, l):
        return self.ws.get(self.lo + t, l)


def _full_and_inputs(sync_op, L=4, D=2):
    wl = I.Workload("tp", T=4, L=L, D=D, hidden=256, heads=4, kv_heads=2, ffn=352, dtype="bf16", mode="prefill", batch=2, seq=300)
    ws = I.WeightSource(wl, gain_jitter=0.1)
    x = I.prefill_inputs(wl)
    xd = I.decode_inputs(wl)
    return wl, ws, x, xd


@pytest.mark.parametrize("sync_op", ["sum", "mean"])
def test_one_rank_with_identity_hook_equals_the_plain_schedule_and_syncs_L_over_D_times(sync_op):
    import torch
    wl, ws, x, xd = _full_and_inputs(sync_op)
    from paper_2602_07306_b200 import pt
    outs = []
    calls = []
    launches = []
    for hooked in (False, True):
        m = Hp.make_model(wl, ws, sync_op=sync_op, max_pos=512)
        if hooked:
            m.set_track_group(wl.T, lambda t: calls.append(t.numel()))
        cache = m.new_cache(2 * 20, 16)
        xdev = Hp.to_dev(m, x)
        n0 = pt.lib().pt_launch_count()
        p = m.prefill(cache, xdev, [0, 1]).cpu().numpy()
        launches.append(pt.lib().pt_launch_count() - n0)
        n_prefill = len(calls)
        d = m.decode_step(cache, Hp.to_dev(m, xd), [0, 1]).cpu().numpy()
        torch.cuda.synchronize()
        assert m.device_status() == (0, 0)
        outs.append((p, d))
        m.close()
    # with a track group a prefill launches, per track block, the kernel that spreads the reduced stream and - except
    # after the last block - the side-stream prefetch of the next layer's QKV weights that runs under the all-reduce
    syncs = wl.L // wl.D
    assert launches[1] - launches[0] == syncs + (syncs - 1)
    # one all-reduce per track block: L/D per forward, against 2L for tensor parallelism
    assert n_prefill == wl.L // wl.D and len(calls) == 2 * (wl.L // wl.D)
    assert calls[0] == 2 * 300 * wl.hidden and calls[-1] == 2 * wl.hidden
    # the two schedules add the partial sums of squares in a different order, which moves a few bf16
    # roundings of the next layer's operands: equal to well inside the bf16 bounds, not bit for bit
    for a, b in zip(outs[0], outs[1]):
        mx, mean = Hp.rel_errs(a, b)
        assert mx <= 1e-2 and mean <= 2.5e-3, (mx, mean)


@pytest.mark.parametrize("sync_op", ["sum", "mean"])
def test_two_ranks_holding_half_the_tracks_each_match_the_single_model(sync_op):
    import torch
    wl, ws, x, xd = _full_and_inputs(sync_op)
    full = Hp.make_model(wl, ws, sync_op=sync_op, max_pos=512)
    cache = full.new_cache(2 * 20, 16)
    want_p = full.prefill(cache, Hp.to_dev(full, x), [0, 1]).cpu().numpy()
    want_d = full.decode_step(cache, Hp.to_dev(full, xd), [0, 1]).cpu().numpy()
    full.close()

    half = I.Workload("half", T=2, L=wl.L, D=wl.D, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads, ffn=wl.ffn,
                      dtype="bf16", mode="prefill", batch=2, seq=300)
    barrier = threading.Barrier(2)
    bufs, results, errors = [None, None], [None, None], []

    def allreduce(rank, t):
        torch.cuda.current_stream().synchronize()          # this rank's partial sum is complete
        bufs[rank] = t
        barrier.wait(timeout=60)
        total = bufs[0] + bufs[1]                           # both ranks add in the same order
        torch.cuda.current_stream().synchronize()
        barrier.wait(timeout=60)                            # nobody overwrites its buffer before both have read
        t.copy_(total)

    def rank_main(rank):
        try:
            with torch.cuda.stream(torch.cuda.Stream()):
                m = Hp.make_model(half, _Tracks(ws, 2 * rank), sync_op=sync_op, max_pos=512)
                m.set_track_group(wl.T, lambda t: allreduce(rank, t))
                c = m.new_cache(2 * 20, 16)
                p = m.prefill(c, Hp.to_dev(m, x[2 * rank:2 * rank + 2]), [0, 1]).cpu().numpy()
                d = m.decode_step(c, Hp.to_dev(m, xd[2 * rank:2 * rank + 2]), [0, 1]).cpu().numpy()
                torch.cuda.current_stream().synchronize()
                assert m.device_status() == (0, 0)
                results[rank] = (p, d)
                m.close()
        except Exception as e:          # a failing rank must not leave the other at the barrier
            errors.append(e)
            barrier.abort()

    threads = [threading.Thread(target=rank_main, args=(r,)) for r in range(2)]
    for th in threads:
        th.start()
    for th in threads:
        th.join(timeout=300)
    assert not errors, errors
    for rank in range(2):
        p, d = results[rank]
        # the ranks add (t0 + t1) + (t2 + t3), the single model ((t0 + t1) + t2) + t3: fp32 rounding only
        # (and a few bf16 roundings downstream of it, as above)
        for got, want in ((p, want_p), (d, want_d)):
            mx, mean = Hp.rel_errs(got, want)
            assert mx <= 1e-2 and mean <= 2.5e-3, (rank, mx, mean)
    assert np.array_equal(results[0][0], results[1][0]) and np.array_equal(results[0][1], results[1][1])
    # and the two-rank result stands on its own against the oracle
    from oracle import pt_oracle as O
    cfg = Hp.oracle_cfg(wl, sync_op)
    ocache = O.PagedKVCache(cfg, 40, 16)
    Hp.assert_close(results[0][0], O.pt_prefill(cfg, ws, x, ocache, [0, 1]), "bf16", "two-rank prefill")
    Hp.assert_close(results[0][1], O.pt_decode_step(cfg, ws, xd, ocache, [0, 1]), "bf16", "two-rank decode")


def test_nccl_all_reduce_as_the_hook_on_a_single_rank_group():
    import os
    import socket
    import torch
    import torch.distributed as dist
    if dist.is_initialized():
        pytest.skip("a process group already exists in this process")
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    dist.init_process_group("nccl", init_method=f"tcp://127.0.0.1:{port}", rank=0, world_size=1, device_id=torch.device("cuda:0"))
    try:
        wl, ws, x, xd = _full_and_inputs("sum")
        plain = Hp.make_model(wl, ws, max_pos=512)
        c0 = plain.new_cache(40, 16)
        want = plain.prefill(c0, Hp.to_dev(plain, x), [0, 1]).cpu().numpy()
        plain.close()
        m = Hp.make_model(wl, ws, max_pos=512)
        m.set_track_group(wl.T, lambda t: dist.all_reduce(t))
        c = m.new_cache(40, 16)
        got = m.prefill(c, Hp.to_dev(m, x), [0, 1]).cpu().numpy()
        torch.cuda.synchronize()
        assert m.device_status() == (0, 0)
        mx, mean = Hp.rel_errs(got, want)
        assert mx <= 1e-2 and mean <= 2.5e-3, (mx, mean)
        m.close()
    finally:
        dist.destroy_process_group()
