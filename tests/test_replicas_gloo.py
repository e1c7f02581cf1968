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


_RANK_PROGRAM = r'''
import json, os, sys
sys.path.insert(0, sys.argv[1])
import torch.distributed as dist
from paper_2607_28150_b200 import replicas
rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
assert os.environ["MASTER_ADDR"] == "127.0.0.1" and int(os.environ["LOCAL_RANK"]) == rank
dist.init_process_group("gloo")
mx = replicas.max_over_ranks({"step": 5.0 + rank})
dist.barrier()
if rank == 0:
    print(json.dumps({"n_gpus": replicas.world(), "ms": mx["step"], "value": replicas.aggregate_throughput(10.0, mx["step"])}))
dist.destroy_process_group()
'''


def test_launcher_starts_one_rank_per_replica_and_returns_rank_zero_output(tmp_path):
    """`bench.py --gpus N` started as a plain process spawns its N ranks with this launcher; here the ranks are CPU
    processes on gloo: both must start, rendezvous on 127.0.0.1, and rank 0's single line must carry world size 2."""
    import json
    import sys
    from paper_2607_28150_b200 import replicas
    prog = tmp_path / "rank.py"
    prog.write_text(_RANK_PROGRAM)
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    codes, out = replicas.launch_local_ranks(2, [sys.executable, str(prog), root], timeout=180)
    assert codes == [0, 0]
    line = json.loads(out.strip().splitlines()[-1])
    assert line == {"n_gpus": 2, "ms": 6.0, "value": 2 * 10.0 / 6.0}
