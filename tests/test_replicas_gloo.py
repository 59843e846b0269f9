"""The N > 1 path of the bench: replicas with a barrier and a max over ranks, here as two gloo ranks on CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), LOCAL_RANK=str(rank), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    from paper_2609_26300_b200.replicas import Replicas
    r = Replicas(backend="gloo")
    r.barrier()
    mine = [100.0 + 7.0 * rank, 50.0 - rank, 3.0]          # per-rank step time, another time, a constant
    got = r.max_over_ranks(mine)
    tps = r.aggregate_tokens_per_s(4, got[0])
    r.barrier()
    out.put((rank, got, tps, r.world))
    r.close()


def test_two_replicas_take_the_max_time_and_sum_the_tokens():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(rk, 2, port, out)) for rk in range(2)]
    for p in procs:
        p.start()
    res = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    for rank, got, tps, world in res:
        assert world == 2
        assert got == [107.0, 50.0, 3.0]                      # slowest rank everywhere
        assert abs(tps - 2 * 4 / 107e-6) < 1e-6 * tps          # both replicas' tokens over the slowest time


def test_single_process_is_a_no_op():
    for k in ("RANK", "WORLD_SIZE", "LOCAL_RANK"):
        os.environ.pop(k, None)
    from paper_2609_26300_b200.replicas import Replicas
    r = Replicas()
    r.barrier()
    assert r.world == 1 and r.max_over_ranks([1.5, 2.5]) == [1.5, 2.5]
    assert r.aggregate_tokens_per_s(4, 100.0) == 4 / 100e-6
