"""The N > 1 path of the benchmark on CPU: two `gloo` ranks.

The PT forward shards over the batch with no data-path collective (batch rows are independent),
so the only things that cross ranks are the timing scalars: the job's step time is the slowest
rank's, its tokens are the sum over ranks.  The reference arm runs on rank 0 alone."""
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
        q.put((rank, out, bench.rank_batch_seed(0, rank)))
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
    for rank, (ms, total, e2e), seed in got:
        assert ms == 12.5                                   # slowest rank
        assert total == 128.0                               # all ranks' tokens
        assert e2e == pytest.approx(128.0 / (64.0 / 4000.0))
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
