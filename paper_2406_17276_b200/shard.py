"""Host-side logic of a multi-process run: one process per GPU, every process builds trees for
its own sequences.  Sequences never exchange data (Algorithm 1 works on one sequence), so there
is no collective on the data path; the processes only meet to time the job: a barrier on both
sides of the timed region, the slowest rank's time, and the number of trees all ranks built.
"""
from __future__ import annotations

from .synth import Workload


def rank_workload(w: Workload, rank: int) -> Workload:
    """The workload of one rank: same shape, its own seed (its own tables and root tokens)."""
    return Workload(**{**w.__dict__, "seed": w.seed + 1000 * rank})


def max_over_ranks(x: float, device: str = "cpu") -> float:
    """The largest x of all ranks (x itself without a process group)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device: str = "cpu") -> float:
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job(units_local: float, ms_local: float, device: str = "cpu") -> tuple[float, float]:
    """(units of all ranks per second, the slowest rank's milliseconds)."""
    ms = max_over_ranks(ms_local, device)
    units = sum_over_ranks(units_local, device)
    return units / (ms * 1e-3), ms


def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launched_by_torchrun() -> bool:
    import os
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ


def launch_ranks(script: str, argv: list[str], nproc: int, port: int | None = None, env: dict | None = None) -> int:
    """Runs `script argv` as nproc ranks on this node (one process per GPU) through torch.distributed.run
    with a loopback rendezvous, and returns the launcher's exit code.  Used when the program was asked
    for several GPUs but was started as a single process."""
    import os
    import subprocess
    import sys
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={nproc}",
           "--master-addr", "127.0.0.1", "--master-port", str(port or free_port()), script, *argv]
    e = dict(os.environ)
    e.update(env or {})
    return subprocess.call(cmd, env=e)


def init_ranks(backend: str, local_device=None):
    """Joins the process group torch.distributed.run set up (rank, world size, local rank from the
    environment); (0, 1, 0) without one."""
    import os
    rank, world = int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1))
    local = int(os.environ.get("LOCAL_RANK", 0))
    if world > 1:
        import torch.distributed as dist
        if local_device is not None:
            dist.init_process_group(backend, device_id=local_device)
        else:
            dist.init_process_group(backend)
    return rank, world, local


class HostTimer:
    """Wall-clock timer with the interface timed_job expects (the device path passes one built on events)."""

    def start(self):
        import time
        self.t0 = time.perf_counter()

    def stop(self):
        import time
        self.t1 = time.perf_counter()

    def elapsed_ms(self) -> float:
        return (self.t1 - self.t0) * 1e3


def timed_job(step, steps: int, warmup: int, units_per_step: float, timer, sync, device: str = "cpu"):
    """The timing protocol of a multi-rank run: `warmup` untimed steps, then exactly `steps` timed steps
    with a barrier and `sync()` on both sides; timer.start() / timer.stop() bracket the steps on this rank
    and timer.elapsed_ms() is read after the closing barrier.  The job's time is the slowest rank's, its
    throughput all ranks' units over that time.  Returns (units per second of the whole job, milliseconds)."""
    import torch.distributed as dist
    grouped = dist.is_available() and dist.is_initialized()

    def fence():
        if grouped:
            dist.barrier()
        sync()

    for i in range(warmup):
        step(i)
    fence()
    timer.start()
    for i in range(steps):
        step(warmup + i)
    timer.stop()
    fence()
    return whole_job(units_per_step * steps, timer.elapsed_ms(), device)
