"""The N > 1 bookkeeping (work partition, barrier, max-over-ranks time, aggregate throughput) on
two CPU ranks over gloo."""
import os

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2609_34606_b200 import sharding


def test_partition_covers_everything_once():
    for n in (0, 1, 7, 30, 31):
        for world in (1, 2, 3, 8):
            spans = [sharding.partition(n, world, r) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == n
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [e - s for s, e in spans]
            assert max(sizes) - min(sizes) <= 1
    assert sharding.assign_layers(30, 8)[0] == [0, 1, 2, 3] and sharding.assign_layers(30, 8)[7] == [27, 28, 29]


def _worker(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    layers = sharding.assign_layers(30, world)[rank]
    dist.barrier()
    # rank 1 is "slower": the job's time is the maximum, its throughput the sum of units over that
    secs = 1.0 + rank
    thr, slow = sharding.aggregate_throughput(units_per_rank=float(len(layers)), seconds_per_rank=secs)
    mx = sharding.max_over_ranks([secs, 10.0 - rank])
    out.put((rank, layers, thr, slow, mx))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_gloo():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + (os.getpid() % 2000)
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, l0, thr0, slow0, mx0), (r1, l1, thr1, slow1, mx1) = res
    assert l0 == list(range(15)) and l1 == list(range(15, 30))
    assert slow0 == slow1 == 2.0 and thr0 == thr1 == 30.0 / 2.0
    assert mx0 == mx1 == [2.0, 10.0]


def test_bench_starts_its_own_ranks():
    """`bench.py --gpus 2` without a launcher starts two ranks itself; with --rank-check they meet over
    gloo, aggregate stand-in numbers (2 units of work over the slower rank's 2 s) and stop before any
    GPU is touched.  A rank count that contradicts the launcher's is refused."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--rank-check"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1 and lines[0]["n_gpus"] == 2 and lines[0]["value"] == 1.0 and lines[0]["slowest_s"] == 2.0
    bad = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "4", "--rank-check"],
                         capture_output=True, text=True, env=dict(env, WORLD_SIZE="2", RANK="0"), timeout=120)
    assert bad.returncode != 0 and "--gpus 4" in bad.stderr
