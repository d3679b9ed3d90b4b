"""The multi-rank bookkeeping on two gloo ranks (CPU): request sharding, slowest-rank time,
whole-job token count and throughput.  Ranks exchange no cache data (each evicts its own
requests), so this is all that N > 1 adds to the single-GPU path."""
import os
import socket

import pytest
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2509_09754_b200 import replicas


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, n_requests, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        mine = replicas.shard_requests(n_requests, rank, world)
        tokens = sum(1000 + 10 * r for r in mine)          # request r has 1000 + 10 r tokens
        ms = 2.0 + rank                                    # rank 1 is the slow one
        out.put((rank, list(mine), replicas.slowest_rank_ms(ms), replicas.whole_job_units(tokens),
                 replicas.whole_job_throughput(tokens, ms)))
        dist.barrier()
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("n_requests", [7, 2, 1])
def test_two_ranks(n_requests):
    world = 2
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_worker, args=(r, world, port, n_requests, out)) for r in range(world)]
    for p in procs:
        p.start()
    got = sorted(out.get(timeout=120) for _ in range(world))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    served = [r for _, mine, _, _, _ in got for r in mine]
    assert served == list(range(n_requests)), "every request is served by exactly one rank"
    assert abs(len(got[0][1]) - len(got[1][1])) <= 1
    total = sum(1000 + 10 * r for r in range(n_requests))
    for _, _, ms, units, thr in got:
        assert ms == 3.0
        assert units == total
        assert thr == pytest.approx(total / 3.0e-3)


def test_single_process_passthrough():
    assert replicas.slowest_rank_ms(1.25) == 1.25
    assert replicas.whole_job_units(77) == 77
    assert list(replicas.shard_requests(5, 0, 1)) == [0, 1, 2, 3, 4]
    with pytest.raises(ValueError):
        replicas.shard_requests(5, 2, 2)
