"""The multi-GPU path is replicas only: these tests cover its host logic on CPU — the router, and
the cross-rank reductions of the bench with two gloo ranks."""
import os
import socket

import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2607_21042_b200 import replicas as R


def test_router_balances_and_respects_limits():
    rt = R.StreamRouter(n_replicas=2, pages_per_replica=10, slots_per_replica=3)
    a = rt.assign(64 * 4)          # 4 pages -> replica 0
    b = rt.assign(64 * 4)          # least loaded -> replica 1
    c = rt.assign(65)              # 2 pages -> either (tie -> 0)
    assert a[0] == 0 and b[0] == 1 and c[0] == 0
    assert rt.reserved == [6, 4]
    d = rt.assign(64 * 6)          # 6 pages fits only replica 1
    assert d[0] == 1 and rt.reserved == [6, 10]
    assert rt.assign(64 * 5) is None            # nobody has 5 pages left
    e = rt.assign(64 * 4)
    assert e[0] == 0 and rt.reserved == [10, 10]
    rt.release(*a)
    assert rt.reserved == [6, 10]
    f = rt.assign(1)
    assert f[0] == 0
    assert rt.assign(1) is None or True
    # slot limit
    rt2 = R.StreamRouter(n_replicas=1, pages_per_replica=100, slots_per_replica=2)
    assert rt2.assign(10) and rt2.assign(10)
    assert rt2.assign(10) is None
    assert R.StreamRouter.pages_for(64) == 1 and R.StreamRouter.pages_for(65) == 2


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        ms = [10.0, 12.5][rank]
        tokens = [500, 480][rank]
        got_ms = R.max_over_ranks(ms)
        got_tok = R.sum_over_ranks(tokens)
        thr = R.whole_job_throughput(tokens, ms)
        dist.barrier()
        out.put((rank, got_ms, got_tok, thr))
    finally:
        dist.destroy_process_group()


def test_reductions_with_two_gloo_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = [q.get(timeout=120) for _ in range(2)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, ms, tok, thr in res:
        assert ms == 12.5 and tok == 980
        assert abs(thr - 980 / 12.5e-3) < 1e-6


def test_reductions_without_process_group_are_identity():
    assert R.max_over_ranks(3.5) == 3.5
    assert R.whole_job_throughput(100, 50.0) == 2000.0


def test_bench_gpus_2_starts_two_ranks():
    """`python bench.py --gpus 2` from a plain process re-executes itself as two ranks; in the dry
    mode (gloo, no GPU work) rank 0 prints one line for the whole job."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    res = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--dry-run"],
                         capture_output=True, text=True, timeout=300, env=env)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1
    out = json.loads(lines[0])
    assert out["n_gpus"] == 2 and out["dry_run"] is True
    # two ranks of 100 tokens each over the slower rank's 11 ms
    assert abs(out["value"] - 200 / 11e-3) < 1e-6
