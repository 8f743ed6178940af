"""Multi-GPU layout of the benchmark: requests are sharded across ranks, nothing is exchanged.

Every step of the path works on independent (request, head) units, so N GPUs serve N times the
requests (weak scaling).  The only communication is the timing reduction: every rank times its own
steps on its device and the job's step time is the maximum over ranks.  Kept free of CUDA so that
the same code runs under the gloo backend on CPU in the tests.
"""
from __future__ import annotations

from . import workloads as wl


def rank_requests(workload: str, rank: int):
    """The requests rank `rank` serves: the workload's request list, re-seeded per rank for the ragged mix."""
    if workload == "cfg1":
        return [dict(family="mamba2", K=8, total=8 * 1024, recompute=1024)]
    if workload == "cfg2":
        return [dict(family="gdn", K=16, total=16 * 1024, recompute=int(0.2 * 16 * 1024))]
    if workload == "cfg3":
        return [dict(family="gdn", K=32, total=32 * 1024, recompute=2048, shared_pool=True) for _ in range(8)]
    if workload == "cfg4":
        return wl.ragged_mix(seed=4 + 1000 * rank)
    raise ValueError(workload)


def job_step_ms(local_ms: float, dist=None, device=None) -> float:
    """Step time of the whole job: the slowest rank's device time (MAX all-reduce), or local_ms alone."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return float(local_ms)
    import torch
    t = torch.tensor([float(local_ms)], dtype=torch.float64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def job_total(local_count: int, dist=None, device=None) -> int:
    """Units (tokens) processed by all ranks together (SUM all-reduce)."""
    if dist is None or not dist.is_initialized() or dist.get_world_size() == 1:
        return int(local_count)
    import torch
    t = torch.tensor([int(local_count)], dtype=torch.int64, device=device if device is not None else "cpu")
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return int(t.item())


def free_port() -> int:
    import socket
    with socket.socket() as sock:
        sock.bind(("127.0.0.1", 0))
        return sock.getsockname()[1]


def launch_ranks(script: str, argv, n: int, timeout=None) -> int:
    """Runs `script argv` as n ranks on this node (torch.distributed.run, rendezvous on 127.0.0.1, a free port):
    RANK / LOCAL_RANK / WORLD_SIZE reach every rank through the environment.  Returns the launcher's exit code;
    the ranks' output goes to this process's stdout / stderr."""
    import subprocess
    import sys
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={int(n)}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), script] + list(argv)
    return subprocess.run(cmd, timeout=timeout).returncode
