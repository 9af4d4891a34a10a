"""World-size-2 gloo test of the replica aggregation used by `bench.py --gpus N` (CPU only)."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2201_05587_b200 import replicas
    r, lr, w = replicas.init("gloo")
    assert (r, w) == (rank, world)
    replicas.barrier()
    # rank 0 does 10 units in 1 s, rank 1 does 10 units in 2 s: 20 units over the slowest rank's 2 s
    value, slowest = replicas.aggregate(10.0, 1.0 + rank)
    out.put((rank, value, slowest, replicas.max_over_ranks(float(rank)), replicas.sum_over_ranks(1.0)))
    replicas.barrier()
    replicas.finalize()


def test_replica_aggregation_world_size_2():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, value, slowest, mx, sm in res:
        assert value == 10.0 and slowest == 2.0 and mx == 1.0 and sm == 2.0


def test_single_process_is_identity():
    from paper_2201_05587_b200 import replicas
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    assert replicas.env_world() == (0, 0, 1)
    assert replicas.aggregate(6.0, 2.0) == (3.0, 2.0)
