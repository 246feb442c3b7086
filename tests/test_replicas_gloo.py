"""The N > 1 mode is N independent replicas: its host logic, run as two gloo ranks on CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp

import kraken_inputs as ki
from paper_2408_07802_b200 import replicas


def _free_port():
    s = socket.socket()
    s.bind(("127.0.0.1", 0))
    p = s.getsockname()[1]
    s.close()
    return p


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), LOCAL_RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    assert replicas.rank_env() == (rank, rank, world)
    dist = replicas.init_process_group("gloo")
    replicas.barrier()
    tok = ki.uniform_tokens(replicas.token_seed(rank), 4096, 1, 64)
    my_ms = 10.0 + 5.0 * rank                     # rank 1 is the slow one
    worst = replicas.max_over_ranks(my_ms)
    value = replicas.whole_job_throughput(64, worst, world)
    gathered = [torch.zeros_like(tok) for _ in range(world)]
    dist.all_gather(gathered, tok)
    out[rank] = (worst, value, bool(torch.equal(gathered[0], gathered[1])))
    replicas.barrier()
    dist.destroy_process_group()


def test_two_replicas_time_is_max_and_throughput_is_whole_job():
    world, port = 2, _free_port()
    with mp.Manager() as mgr:
        out = mgr.dict()
        mp.spawn(_worker, args=(world, port, out), nprocs=world, join=True)
        res = dict(out)
    for rank in range(world):
        worst, value, same_tokens = res[rank]
        assert worst == 15.0                                  # max over ranks, on every rank
        assert abs(value - 2 * 64 / 15e-3) < 1e-6             # all ranks' tokens over the slowest time
        assert not same_tokens                                # replicas serve different requests


def test_single_process_defaults():
    for k in ("RANK", "LOCAL_RANK", "WORLD_SIZE"):
        os.environ.pop(k, None)
    assert replicas.rank_env() == (0, 0, 1)
    assert replicas.max_over_ranks(3.5) == 3.5
    assert replicas.whole_job_throughput(100, 50.0, 1) == 2000.0
