"""Host-side helpers for running N independent replicas of the path (one process per GPU).

The path shards with no exchange (independent per layer, sequence and KV head), so multi-GPU runs are
replicas: torch.distributed is used only for a barrier and to take the maximum of the device times over
ranks.  No data-path collective exists."""
from __future__ import annotations

from typing import Dict

import torch.distributed as dist


def world() -> int:
    return dist.get_world_size() if dist.is_available() and dist.is_initialized() else 1


def max_over_ranks(times: Dict[str, float]) -> Dict[str, float]:
    """Element-wise maximum of a dict of per-stage times over all ranks (identity for one process)."""
    if world() == 1:
        return dict(times)
    gathered = [None] * world()
    dist.all_gather_object(gathered, times)
    return {k: max(g[k] for g in gathered) for k in times}


def aggregate_throughput(units_per_rank: float, seconds_max_over_ranks: float) -> float:
    """Whole-job throughput of `world()` replicas that each processed `units_per_rank` in the given time."""
    return world() * units_per_rank / seconds_max_over_ranks


def free_port() -> int:
    import socket
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def launch_local_ranks(n: int, argv, env=None, timeout=None):
    """Start `n` copies of the command `argv` on this node, one per rank, with the rendezvous variables
    torch.distributed reads (RANK, LOCAL_RANK, WORLD_SIZE, MASTER_ADDR = 127.0.0.1, MASTER_PORT), wait for all
    of them and return (exit codes, stdout of rank 0).  This is what `bench.py --gpus N` does when it is started
    as a plain process instead of under torchrun: the replicas exchange nothing but a barrier and a maximum."""
    import os
    import subprocess
    port = free_port()
    procs = []
    for r in range(n):
        e = dict(os.environ if env is None else env)
        e.update(RANK=str(r), LOCAL_RANK=str(r), WORLD_SIZE=str(n), MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        procs.append(subprocess.Popen(list(argv), env=e, stdout=subprocess.PIPE if r == 0 else subprocess.DEVNULL))
    out0 = procs[0].communicate(timeout=timeout)[0]
    codes = [procs[0].returncode] + [p.wait(timeout=timeout) for p in procs[1:]]
    return codes, (out0 or b"").decode()
