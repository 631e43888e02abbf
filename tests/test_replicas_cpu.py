"""The benchmark's multi-rank bookkeeping on CPU: two gloo ranks, max-over-ranks time and
summed work.  (The path itself does not shard: N GPUs run N replicas.)"""
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
    from paper_2602_12305_b200 import replicas
    r, w = replicas.init("gloo")
    assert (r, w) == (rank, world)
    replicas.barrier()
    ms, units = replicas.aggregate(10.0 + 5.0 * rank, 3.0 + rank)     # rank 1 is slower and did more
    assert replicas.any_rank(rank == 1) is True and replicas.any_rank(False) is False
    out.put((rank, ms, units))
    replicas.barrier()
    replicas.shutdown()


def test_two_rank_aggregate_is_max_time_and_summed_work():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert got == [(0, 15.0, 7.0), (1, 15.0, 7.0)]


def test_single_process_is_a_pass_through(monkeypatch):
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        monkeypatch.delenv(k, raising=False)
    from paper_2602_12305_b200 import replicas
    assert replicas.env_world() == (0, 0, 1)
    assert replicas.init("gloo") == (0, 1)
    replicas.barrier()
    assert replicas.aggregate(2.5, 4.0) == (2.5, 4.0)
    assert replicas.any_rank(True) is True and replicas.any_rank(False) is False
