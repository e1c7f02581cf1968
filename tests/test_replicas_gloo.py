"""World-size-2 gloo test of the replica aggregation used by `bench.py --gpus N` (runs on CPU)."""
import os
import socket

import torch.distributed as dist
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank), WORLD_SIZE=str(world))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    from paper_2607_28150_b200 import replicas
    times = {"select": 1.0 + rank, "pack": 2.0 - rank, "decode": 10.0 * (rank + 1)}
    mx = replicas.max_over_ranks(times)
    dist.barrier()
    q.put((rank, mx, replicas.aggregate_throughput(100.0, mx["decode"]), replicas.world()))
    dist.destroy_process_group()


def test_max_over_ranks_and_aggregate_throughput_two_ranks():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in procs]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, mx, thr, w in got:
        assert w == 2
        assert mx == {"select": 2.0, "pack": 2.0, "decode": 20.0}
        assert thr == 2 * 100.0 / 20.0


def test_single_process_is_identity():
    from paper_2607_28150_b200 import replicas
    assert replicas.max_over_ranks({"a": 3.0}) == {"a": 3.0}
    assert replicas.aggregate_throughput(10.0, 2.0) == 5.0
