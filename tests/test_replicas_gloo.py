"""The multi-GPU mode is N independent replicas; only the timing is reduced.  Two gloo ranks on CPU."""
import os
import socket

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2606_17421_b200.replicas import job_ms_per_token, max_over_ranks


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _rank_main(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    mine = 2.0 + 3.0 * rank                      # rank 1 is the slow one
    slowest = max_over_ranks(mine)
    dist.barrier()
    out.put((rank, slowest, job_ms_per_token(slowest, world)))
    dist.destroy_process_group()


def test_timing_reduction_over_two_ranks():
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    results = sorted(out.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results == [(0, 5.0, 2.5), (1, 5.0, 2.5)]


def test_single_process_is_a_no_op():
    assert max_over_ranks(3.25) == 3.25
    assert job_ms_per_token(3.0, 1) == 3.0
