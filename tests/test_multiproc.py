"""The N > 1 paths on CPU: two `gloo` ranks.

The PT forward shards over the batch with no data-path collective (batch rows are independent),
so the only things that cross ranks are the timing scalars: the job's step time is the slowest
rank's, its tokens are the sum over ranks.  The reference arm runs on rank 0 alone.  With tracks
split over ranks (Section 2.2's placement) the data path has one exchange, an all-reduce per track
block: the last test runs that decomposition through a real all-reduce with the oracle as each
rank's compute."""
import json
import os
import socket
import subprocess
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        ms = [10.0, 12.5][rank]                  # rank 1 is the slow one
        tokens = [64.0, 64.0][rank]
        e2e = [6000.0, 4000.0][rank]             # tokens/s end to end: 64/6000 s and 64/4000 s per step
        out = bench.aggregate_over_ranks(ms, tokens, e2e, world, torch.device("cpu"))
        tr = bench.aggregate_track_ranks(ms, tokens, e2e, world, torch.device("cpu"))
        q.put((rank, out, bench.rank_batch_seed(0, rank), tr))
    finally:
        dist.destroy_process_group()


def test_two_gloo_ranks_aggregate_max_time_and_sum_tokens():
    import torch.multiprocessing as mp
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, (ms, total, e2e), seed, tr in got:
        assert ms == 12.5                                   # slowest rank
        assert total == 128.0                               # all ranks' tokens
        assert e2e == pytest.approx(128.0 / (64.0 / 4000.0))
        # tracks split over the ranks: one batch for the whole job, the slowest rank's time
        assert tr[0] == 12.5 and tr[1] == 64.0 and tr[2] == pytest.approx(64.0 / (64.0 / 4000.0))
    assert got[0][2] != got[1][2]                           # each rank draws its own batch


def test_single_rank_aggregate_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.aggregate_over_ranks(3.0, 64, 100.0, 1, None) == (3.0, 64.0, 100.0)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--steps", "1", "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_reference_arm_prints_one_json_line_with_the_oracle_baseline():
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--workload", "cfg1",
                        "--steps", "1", "--warmup", "0"], capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-500:]
    line = json.loads(r.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["value"] > 0 and line["unit"] == "tokens/s"
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] >= 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["e2e"]["d2h_bytes_per_step"] == 0


class _Sub:
    """Weights of tracks [t_lo, ...) and layers [l_lo, ...) of a larger stack, renumbered from 0."""
    def __init__(self, ws, t_lo, l_lo):
        self.ws, self.t_lo, self.l_lo = ws, t_lo, l_lo

    def get(self, t, l):
        return self.ws.get(self.t_lo + t, self.l_lo + l)


def _track_rank(rank, world, port, sync_op, q):
    """One rank of a track group on CPU: its share of the tracks through the oracle, block by block,
    with one gloo all-reduce of the partial sum per track block."""
    import numpy as np
    import torch
    import torch.distributed as dist
    sys.path.insert(0, ROOT)
    from oracle import pt_oracle as O
    from paper_2602_07306_b200 import inputs as I
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        wl = I.Workload("tp-cpu", T=4, L=4, D=2, hidden=64, heads=2, kv_heads=1, ffn=96, dtype="fp32", mode="prefill", batch=2, seq=9)
        ws = I.WeightSource(wl, gain_jitter=0.1)
        x = I.prefill_inputs(wl).astype(np.float64)                          # [T, B, S, H]
        per = wl.T // world
        block = O.PTConfig(T=per, D=wl.D, L=wl.D, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads, ffn=wl.ffn,
                           rope_base=wl.rope_base, rms_eps=wl.rms_eps, sync_op="sum")
        xin, n_collectives = x[rank * per:(rank + 1) * per], 0
        for b in range(wl.L // wl.D):
            cache = O.PagedKVCache(block, wl.batch * 1, 16)
            part = O.pt_prefill(block, _Sub(ws, rank * per, b * wl.D), xin, cache, list(range(wl.batch)), None)   # sum of this rank's tracks
            t = torch.from_numpy(np.ascontiguousarray(part))
            dist.all_reduce(t)                                               # the one exchange of the block
            n_collectives += 1
            h = t.numpy() / (wl.T if sync_op == "mean" else 1)
            xin = np.broadcast_to(h, (per,) + h.shape)                       # every local track continues from the synced stream
        q.put((rank, h, n_collectives))
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("sync_op", ["sum", "mean"])
def test_tracks_split_over_two_gloo_ranks_with_one_all_reduce_per_block_equal_the_whole_model(sync_op):
    import numpy as np
    import torch.multiprocessing as mp
    sys.path.insert(0, ROOT)
    from oracle import pt_oracle as O
    from paper_2602_07306_b200 import inputs as I
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_track_rank, args=(r, 2, port, sync_op, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted((q.get(timeout=180) for _ in procs), key=lambda g: g[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    wl = I.Workload("tp-cpu", T=4, L=4, D=2, hidden=64, heads=2, kv_heads=1, ffn=96, dtype="fp32", mode="prefill", batch=2, seq=9)
    ws = I.WeightSource(wl, gain_jitter=0.1)
    cfg = O.PTConfig(T=wl.T, D=wl.D, L=wl.L, hidden=wl.hidden, heads=wl.heads, kv_heads=wl.kv_heads, ffn=wl.ffn,
                     rope_base=wl.rope_base, rms_eps=wl.rms_eps, sync_op=sync_op)
    cache = O.PagedKVCache(cfg, wl.batch, 16)
    want = O.pt_prefill(cfg, ws, I.prefill_inputs(wl).astype(np.float64), cache, list(range(wl.batch)), None)
    for rank, h, n in got:
        assert n == wl.L // wl.D                            # L/D exchanges per forward (tensor parallelism: 2L)
        assert np.allclose(h, want, rtol=1e-11, atol=1e-12), (rank, float(np.abs(h - want).max()))
    assert np.array_equal(got[0][1], got[1][1])
