"""Process-group plumbing of the benchmark: one process per GPU, partitions with no data-path collective.

Only the barrier, the max-over-ranks of a time and the aggregation of the per-rank work cross
ranks.  The functions are backend-agnostic (NCCL on GPUs, gloo in the CPU tests).
"""
import os
import socket
import subprocess
import sys

import torch


def env_world():
    """(rank, world_size, local_rank) from the launcher's environment (1 process when absent)."""
    return int(os.environ.get("RANK", 0)), int(os.environ.get("WORLD_SIZE", 1)), int(os.environ.get("LOCAL_RANK", 0))


class Group:
    """Thin wrapper: a no-op for one process, torch.distributed otherwise."""

    def __init__(self, backend=None, device=None):
        self.rank, self.world, self.local = env_world()
        self.device = device if device is not None else torch.device("cpu")
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            kw = {}
            if backend == "nccl":
                kw["device_id"] = self.device
            dist.init_process_group(backend, **kw)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()
        if self.device.type == "cuda":
            torch.cuda.synchronize(self.device)

    def max_over_ranks(self, x: float) -> float:
        """Slowest rank's time: the whole job is as slow as its slowest partition."""
        if self.dist is None:
            return float(x)
        t = torch.tensor([float(x)], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return float(t.item())

    def sum_over_ranks(self, x: float) -> float:
        if self.dist is None:
            return float(x)
        t = torch.tensor([float(x)], dtype=torch.float64, device=self.device)
        self.dist.all_reduce(t, op=self.dist.ReduceOp.SUM)
        return float(t.item())

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()


def job_throughput(units_per_rank: float, ms_per_step_local: float, group: Group):
    """Whole-job throughput of a partitioned run: units of ALL ranks per second of the SLOWEST rank.
    Returns (units_per_second, ms_per_step_max)."""
    ms = group.max_over_ranks(ms_per_step_local)
    total_units = group.sum_over_ranks(units_per_rank)
    return total_units / (ms * 1e-3), ms


def shard(items, rank, world):
    """Contiguous shard of a list of independent work items for one rank (sizes differ by at most one)."""
    n = len(items)
    lo, hi = (n * rank) // world, (n * (rank + 1)) // world
    return items[lo:hi]


def free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    port = s.getsockname()[1]
    s.close()
    return port


def spawn_ranks(nproc, argv, extra_env=None, timeout=None):
    """Runs `argv` (a command line) as `nproc` ranks on this node, one process per GPU: RANK = LOCAL_RANK = 0..nproc-1,
    WORLD_SIZE, MASTER_ADDR = 127.0.0.1 and a free MASTER_PORT in the environment -- what a launcher would set.  The
    children inherit stdout / stderr (rank 0 prints the result line).  Returns the largest exit code; if a rank
    fails the others are terminated (by their own PIDs)."""
    port = free_port()
    procs = []
    for r in range(nproc):
        env = dict(os.environ, RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(nproc), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        if extra_env:
            env.update(extra_env)
        procs.append(subprocess.Popen(list(argv), env=env))
    worst, pending = 0, set(range(nproc))
    import time
    t0 = time.monotonic()
    while pending:
        for r in sorted(pending):
            rc = procs[r].poll()
            if rc is not None:
                pending.discard(r)
                worst = max(worst, abs(rc))
        if worst or (timeout is not None and time.monotonic() - t0 > timeout):
            for r in pending:
                procs[r].terminate()
            for r in pending:
                try:
                    procs[r].wait(timeout=10)
                except subprocess.TimeoutExpired:
                    procs[r].kill()
            return worst or 124
        time.sleep(0.05)
    return worst


def launched_by_a_launcher():
    return "WORLD_SIZE" in os.environ and "RANK" in os.environ
