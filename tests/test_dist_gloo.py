"""World-size-2 check (gloo, CPU) of the replica plumbing: rendezvous from the
environment, barrier, and the sum-of-units / max-of-time reduction."""
import os
import socket

import torch.multiprocessing as mp


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2602_14338_b200 import dist as D
    import torch.distributed as dist

    r, w, _ = D.init_from_env("gloo")
    D.barrier()
    units, ms = D.aggregate(100.0 * (r + 1), 10.0 + 5.0 * r)
    q.put((r, w, units, ms))
    D.barrier()
    dist.destroy_process_group()


def test_two_rank_aggregate():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(60)
        assert p.exitcode == 0
    assert [g[0] for g in got] == [0, 1] and all(g[1] == 2 for g in got)
    assert all(g[2] == 300.0 and g[3] == 15.0 for g in got)


def test_single_process_passthrough():
    from paper_2602_14338_b200 import dist as D

    assert D.aggregate(7.0, 3.5) == (7.0, 3.5)
