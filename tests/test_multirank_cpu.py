"""The N > 1 path of the benchmark on CPU: two gloo ranks, request sharding and the timing reduction."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2608_11231_b200 import sharding


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    reqs = sharding.rank_requests("cfg4", rank)
    tokens = sum(r["total"] for r in reqs)
    local_ms = 10.0 + 5.0 * rank                      # rank 1 is the slow one
    step = sharding.job_step_ms(local_ms, dist)
    total = sharding.job_total(tokens, dist)
    out.put((rank, tokens, step, total, [r["K"] for r in reqs][:4]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_ranks_shard_requests_and_reduce_time():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    (r0, tok0, step0, total0, k0), (r1, tok1, step1, total1, k1) = res
    assert step0 == step1 == 15.0                      # max over ranks
    assert total0 == total1 == tok0 + tok1             # whole-job units
    assert k0 != k1                                    # each rank serves its own seeded requests
    assert all(8192 <= r["total"] <= 32768 for r in sharding.rank_requests("cfg4", 1))


def test_single_rank_needs_no_process_group():
    assert sharding.job_step_ms(3.5) == 3.5 and sharding.job_total(7) == 7
    assert len(sharding.rank_requests("cfg3", 0)) == 8


def test_bench_launches_its_own_ranks():
    """`bench.py --gpus 2` started as a plain script becomes the launcher of two ranks; with --dry-run the ranks are
    gloo processes on CPU with a stand-in step (rank r sleeps r + 1 ms), everything else is the benchmark's own path."""
    import json
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items() if k not in ("WORLD_SIZE", "RANK", "LOCAL_RANK")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--gpus", "2", "--steps", "5", "--warmup", "1",
                        "--dry-run"], capture_output=True, text=True, timeout=300, env=env)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [ln for ln in r.stdout.splitlines() if ln.startswith("{")]
    assert len(lines) == 1                               # rank 0 alone prints
    line = json.loads(lines[0])
    tokens = sum(q["total"] for rank in range(2) for q in sharding.rank_requests("cfg4", rank))
    assert line["n_gpus"] == 2 and line["config"]["context_tokens"] == tokens
    assert line["ms_per_step"] >= 2.0                    # the slow rank's time, not rank 0's
    assert abs(line["value"] - tokens / (line["ms_per_step"] * 1e-3)) <= 1e-6 * line["value"]
