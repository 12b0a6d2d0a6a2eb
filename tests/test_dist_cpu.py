"""world_size-2 CPU check (gloo) of the benchmark's multi-rank plumbing: every rank draws its own
request, nothing of the data path is exchanged, the timed region is bracketed by barriers and the
reported time is the maximum over ranks."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2609_07008_b200 import dist as rkdist
from paper_2609_07008_b200 import synth


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, w, _ = rkdist.init("gloo")
    assert (r, w) == (rank, world)
    prof, lay, prot = synth.make_geometry("tiny")
    wl = synth.make_tensors("tiny", prof, lay, prot, rkdist.rank_seed(synth.CONFIGS["tiny"]["seed"], rank))
    rkdist.barrier()
    my_seconds = 0.010 * (rank + 1)                 # stand-in for this rank's device time
    slowest = rkdist.max_over_ranks(my_seconds)
    rkdist.barrier()
    out.put((rank, float(wl.kv.float().sum()), slowest,
             rkdist.aggregate_throughput(lay.n_rows, 5, world, slowest)))
    rkdist.shutdown()


def test_two_ranks_independent_requests_and_max_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, s0, t0, v0), (r1, s1, t1, v1) = res
    assert s0 != s1                                  # different request values per rank
    assert t0 == t1 == 0.020                         # both see the slowest rank's time
    assert v0 == v1 == 2 * 576 * 5 / 0.020           # whole-job throughput over the slowest time


def test_single_rank_is_a_noop():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert rkdist.init("gloo") == (0, 1, 0)
    rkdist.barrier()
    assert rkdist.max_over_ranks(1.5) == 1.5
    assert rkdist.aggregate_throughput(100, 3, 1, 2.0) == 150.0


def test_bench_starts_its_own_ranks_when_launched_plainly():
    """`python bench.py --gpus 2` without a launcher around it starts two ranks itself; on the checker arm
    (no GPU needed) rank 0 alone does the work and exactly one JSON line with n_gpus = 2 comes out."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--impl", "reference", "--config", "tiny",
                        "--steps", "1", "--warmup", "0", "--oracle-pairs", "100000"], capture_output=True, text=True,
                       timeout=600, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [l for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["n_gpus"] == 2 and d["impl"] == "reference" and d["config"]["workload"] == "tiny"
