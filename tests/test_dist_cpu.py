"""The multi-process plumbing of the benchmark (replicas, max over ranks) on CPU with gloo, world size 2."""
import os
import socket

import torch.multiprocessing as mp


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank: int, world: int, port: int, q):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2607_08973_b200 import dist
    r, w, local = dist.init_from_env(world, backend="gloo")
    dist.barrier()
    slowest = dist.max_over_ranks(1.5 + rank)          # rank 1 is the slow replica
    total = dist.sum_over_ranks(10.0 * (rank + 1))
    dist.finalize()
    q.put((r, w, local, slowest, total))


def test_two_replicas_report_the_slowest_rank():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[:3] for g in got] == [(0, 2, 0), (1, 2, 1)]
    assert all(g[3] == 2.5 and g[4] == 30.0 for g in got)


def test_single_process_needs_no_process_group():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    from paper_2607_08973_b200 import dist
    assert dist.init_from_env(1) == (0, 1, 0)
    assert dist.max_over_ranks(3.25) == 3.25
    dist.barrier()
    dist.finalize()


def test_world_size_mismatch_is_refused():
    import pytest
    from paper_2607_08973_b200 import dist
    os.environ.pop("WORLD_SIZE", None)
    with pytest.raises(RuntimeError):
        dist.init_from_env(2)
