"""The N>1 path (token sharding + max-over-ranks timing) on two gloo ranks on the CPU."""
import os
import socket

import torch
import torch.multiprocessing as mp

from paper_2510_11370_b200 import dist as r3dist


def test_shard_ranges_cover_everything_once():
    for total in (0, 1, 7, 4096, 4097):
        for world in (1, 2, 3, 8):
            spans = [r3dist.shard_range(total, r, world) for r in range(world)]
            assert spans[0][0] == 0 and spans[-1][1] == total
            assert all(a[1] == b[0] for a, b in zip(spans, spans[1:]))
            sizes = [hi - lo for lo, hi in spans]
            assert max(sizes) - min(sizes) <= 1


def _worker(rank, world, port, out):
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    r, w = r3dist.init("gloo")
    lo, hi = r3dist.shard_range(1001, r, w)
    r3dist.barrier()
    slowest = r3dist.max_over_ranks(10.0 + r)           # rank 1 is "slower"
    units = r3dist.sum_over_ranks(hi - lo)
    out.put((r, slowest, units))
    torch.distributed.destroy_process_group()


def test_two_ranks_agree_on_job_time_and_total_units():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [r[0] for r in res] == [0, 1]
    assert all(r[1] == 11.0 and r[2] == 1001.0 for r in res)
