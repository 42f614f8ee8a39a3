"""Rank bookkeeping for bench.py: the hot path has no exchange step, so N GPUs run N independent
replicas; the only collective work is the barrier around the timed region and the max-over-ranks
of the measured times.  Backend: nccl on GPUs, gloo in the CPU tests."""
from __future__ import annotations

import os
from typing import Sequence

import torch
import torch.distributed as dist


def env_rank():
    return int(os.environ.get("RANK", "0")), int(os.environ.get("WORLD_SIZE", "1")), int(os.environ.get("LOCAL_RANK", "0"))


def init(backend: str, device=None):
    """Initialises the default process group from the torchrun environment when WORLD_SIZE > 1."""
    rank, world, _ = env_rank()
    if world > 1 and not dist.is_initialized():
        kw = {"device_id": device} if (backend == "nccl" and device is not None) else {}
        dist.init_process_group(backend, rank=rank, world_size=world, **kw)
    return rank, world


def barrier(device=None):
    if dist.is_available() and dist.is_initialized():
        dist.barrier()


def max_over_ranks(values: Sequence[float], device="cpu") -> list:
    """Element-wise maximum of a short list of floats over all ranks (identity for one rank)."""
    t = torch.tensor(list(values), dtype=torch.float64, device=device)
    if dist.is_available() and dist.is_initialized() and dist.get_world_size() > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return [float(x) for x in t]


def replica_throughput(units_per_replica: float, ms_max: float, world: int) -> float:
    """Whole-job throughput of `world` independent replicas that all finished within ms_max."""
    return world * units_per_replica / (ms_max * 1e-3)


def launched_by_torchrun() -> bool:
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def spawn_replicas(argv: Sequence[str], world: int, timeout_s: float = 3600.0) -> int:
    """Starts `world` copies of `argv` (a full command line), one per rank, with the torchrun environment
    (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR=127.0.0.1, a free MASTER_PORT) and waits for them.  All ranks
    inherit stdout/stderr; only rank 0 prints the result line.  Returns the largest exit code; if one rank
    fails the others are terminated (each is a child this function started, addressed by its own pid)."""
    import socket
    import subprocess
    import time
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    procs = []
    for r in range(world):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                   MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=env))
    deadline = time.time() + timeout_s
    code = 0
    alive = list(procs)
    while alive:
        for p in list(alive):
            rc = p.poll()
            if rc is not None:
                alive.remove(p)
                code = max(code, abs(rc))
        if (code != 0 or time.time() > deadline) and alive:
            for p in alive:
                p.terminate()
            for p in alive:
                try:
                    p.wait(timeout=10)
                except subprocess.TimeoutExpired:
                    p.kill()
            return code if code != 0 else 124
        time.sleep(0.05)
    return code


def shutdown():
    if dist.is_available() and dist.is_initialized():
        dist.destroy_process_group()
