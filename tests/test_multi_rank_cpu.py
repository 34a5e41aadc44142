"""The N > 1 path of bench.py on CPU: two gloo ranks, no GPU.

The hot path shards over (batch, head) with no exchange, so the only multi-rank logic is: every rank draws its own
seeded batch, times itself, and the job's throughput is all tokens over the slowest rank's time.  The oracle stands
in for the device step here (tiny shapes)."""
import os
import sys

import numpy as np
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)


def _rank(rank, world, port, out):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    import bench
    from oracle import oracle
    from paper_2608_21308_b200 import inputs
    dist.init_process_group("gloo", rank=rank, world_size=world)
    r = inputs.Recipe(B=1, H=2, L=16, d=4, h=8, C=4)
    x = inputs.generate(bench.shard_recipe(r, rank))
    res = oracle.forward(x["q"], x["k"], x["v"], x["eta"], x["beta"], x["gamma"], x["W"], None, r.C, r.kind, threads=1)
    ms = 10.0 * (rank + 1)                       # pretend device times: rank 1 is the slow one
    ms_max = bench.max_over_ranks(ms, dist, "cpu")
    dist.barrier()
    out.put((rank, float(np.sum(res["o"])), float(x["q"].sum()), ms_max, bench.whole_job_value(world, r.B * r.L, ms_max)))
    dist.destroy_process_group()


def test_two_ranks_independent_shards_and_max_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = 29500 + os.getpid() % 1000
    procs = [ctx.Process(target=_rank, args=(i, 2, port, out)) for i in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, o0, q0, m0, v0), (r1, o1, q1, m1, v1) = got
    assert q0 != q1 and o0 != o1                 # every rank has its own batch
    assert m0 == m1 == 20.0                      # MAX over ranks
    assert v0 == v1 == 2 * 16 / 20e-3            # all tokens / slowest time


def test_bench_gpus_flag_starts_its_own_ranks():
    """`python bench.py --gpus 2` (no torchrun around it) must start two ranks itself; --rank-check makes them meet on
    gloo without touching a GPU and rank 0 report what it saw."""
    import json
    import subprocess
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--gpus", "2", "--rank-check"], env=env,
                         capture_output=True, text=True, timeout=300)
    assert out.returncode == 0, out.stderr[-2000:]
    line = [ln for ln in out.stdout.splitlines() if ln.startswith("{")][-1]
    rec = json.loads(line)
    assert rec["world"] == 2 and rec["ranks_seen"] == 2 and rec["n_gpus"] == 2
