"""world_size-2 gloo test of the replica aggregation (sum of units, max of time)."""
import os
import socket

import pytest

torch = pytest.importorskip("torch")
import torch.multiprocessing as mp  # noqa: E402


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, q):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world),
                      MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    from paper_2609_33385_b200 import dist as d
    r, lr, w = d.init("gloo")
    d.barrier()
    units, ms = d.aggregate(100.0 * (rank + 1), 10.0 + 5.0 * rank)
    q.put((r, w, units, ms))
    d.shutdown()


def test_aggregate_sum_units_max_time_two_ranks():
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
    assert [r[0] for r in res] == [0, 1] and all(r[1] == 2 for r in res)
    assert all(r[2] == 300.0 and r[3] == 15.0 for r in res)


def test_aggregate_single_process_is_identity():
    from paper_2609_33385_b200 import dist as d
    assert d.aggregate(7.0, 3.5) == (7.0, 3.5)
