"""The N > 1 path of the benchmark on CPU: two gloo ranks, independent shards,
throughput = units summed over ranks / time maxed over ranks."""
import os
import socket

import torch.multiprocessing as mp

from paper_2512_20687_b200 import workloads as wl


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2512_20687_b200 import dist as pd
    r, lr, w = pd.init("gloo")
    lo, hi = wl.shard_units(101, w, r)
    pd.barrier()
    mx = pd.reduce_max(1.0 + r)                # rank 1 is the slow one
    total = pd.reduce_sum(hi - lo)
    thr = pd.job_throughput(hi - lo, 1.0 + r)
    pd.barrier()
    pd.shutdown()
    q.put((r, lo, hi, mx, total, thr))


def test_two_gloo_ranks_reduce_time_by_max_and_units_by_sum():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [(r[1], r[2]) for r in res] == [(0, 51), (51, 101)]
    for r in res:
        assert r[3] == 2.0 and r[4] == 101.0 and abs(r[5] - 101.0 / 2.0) < 1e-12


def test_bench_starts_its_own_ranks_when_no_launcher_did():
    """`bench.py --gpus N` started plainly launches N ranks of itself; here through the CPU arm of the script
    (the oracle on the tiny workload), which rank 0 alone runs while the other rank exits 0: one JSON line,
    and it names both ranks."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    code = ("import sys, bench; sys.exit(bench.spawn_ranks(2, ['--impl', 'reference', '--gpus', '2', '--config', '0', "
            "'--steps', '1', '--warmup', '0']))")
    env = {k: v for k, v in os.environ.items() if k not in ("RANK", "LOCAL_RANK", "WORLD_SIZE", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, "-c", code], cwd=root, env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    assert lines[0]["impl"] == "reference" and lines[0]["n_gpus"] == 2 and lines[0]["value"] > 0
