"""The N > 1 launch path on CPU: two gloo ranks shard a batch, agree on the
slowest rank's time and on the whole-job rate."""
import os
import socket

import pytest
import torch
import torch.multiprocessing as mp

from paper_2405_12532_b200 import dist as pdist
from paper_2405_12532_b200 import synth


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    r, w, lr = pdist.env_rank_world()
    assert (r, w, lr) == (rank, world, rank)
    pdist.init("gloo")
    lo, hi = synth.shard_batch(10, w, r)
    pdist.barrier(w)
    mine = [0.5 + 0.25 * r, 2.0 - r]          # rank 1 is slower on the first, faster on the second
    mx = pdist.max_over_ranks(mine, w)
    gathered = [None] * w
    torch.distributed.all_gather_object(gathered, (lo, hi))
    if r == 0:
        out.put((mx, gathered, pdist.whole_job_rate(100.0, w, mx[0])))
    pdist.barrier(w)
    torch.distributed.destroy_process_group()


def test_two_gloo_ranks_agree_on_time_and_rate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    mx, spans, rate = q.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert mx == [0.75, 2.0]
    assert spans == [(0, 5), (5, 10)]          # the shards tile the batch
    assert rate == pytest.approx(2 * 100.0 / 0.75)


def test_single_rank_needs_no_process_group():
    assert pdist.max_over_ranks([1.5, 0.25], 1) == [1.5, 0.25]
    assert pdist.whole_job_rate(64 * 2048, 1, 0.1) == pytest.approx(64 * 2048 / 0.1)


def test_bench_gpus_flag_starts_that_many_ranks():
    """`bench.py --gpus 2` outside a launcher starts two ranks itself; its dry run goes through the
    same rendezvous, barrier and max-over-ranks as the timed run, on gloo, and prints one line."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--dry-run"], env=env,
                       capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["slowest_rank_seconds"] == 2.0 and out["rank0_sequences"] == [0, 64]
