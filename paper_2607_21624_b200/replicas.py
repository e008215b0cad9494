"""Replica bookkeeping for runs on several GPUs of one node.

The layer step does not shard: every rank runs the same workload on its own GPU and no
tensor of the data path crosses ranks.  The only communication is for measurement: a
barrier on both sides of the timed region and the maximum over ranks of the per-step
time, from which the whole-job throughput is derived.
"""
from __future__ import annotations

import os


class Replicas:
    def __init__(self, backend: str = "nccl", device=None):
        self.rank = int(os.environ.get("RANK", "0"))
        self.local_rank = int(os.environ.get("LOCAL_RANK", "0"))
        self.world = int(os.environ.get("WORLD_SIZE", "1"))
        self.device = device
        self.dist = None
        if self.world > 1:
            import torch.distributed as dist
            kw = {}
            if backend == "nccl" and device is not None:
                kw["device_id"] = device
            dist.init_process_group(backend, **kw)
            self.dist = dist

    def barrier(self):
        if self.dist is not None:
            self.dist.barrier()

    def max_over_ranks(self, values):
        """Element-wise maximum over ranks of a list of floats (every rank gets the result)."""
        if self.dist is None:
            return [float(v) for v in values]
        import torch
        t = torch.tensor(list(values), dtype=torch.float64, device=self.device if self.device is not None else "cpu")
        if t.device.type == "cuda":
            t = t.float()
        self.dist.all_reduce(t, op=self.dist.ReduceOp.MAX)
        return [float(v) for v in t.cpu()]

    def whole_job_rate(self, units_per_rank: float, ms_per_step: float) -> float:
        """Units per second of all replicas together, given the slowest rank's time per step."""
        return self.world * units_per_rank / (ms_per_step * 1e-3)

    def close(self):
        if self.dist is not None:
            self.dist.destroy_process_group()
            self.dist = None


def _replica_entry(rank, world, port, fn, args):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    fn(*args)


def spawn_replicas(world: int, fn, *args):
    """Run ``fn(*args)`` in ``world`` fresh processes, one per replica, each with the rank variables a launcher
    would have set (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, a free MASTER_PORT), and wait for all
    of them.  ``fn`` must be importable from the child (a module-level function).  Used by a command that is
    asked for several GPUs without having been started under a launcher."""
    import socket

    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    mp.spawn(_replica_entry, args=(world, port, fn, args), nprocs=world, join=True)
