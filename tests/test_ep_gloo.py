"""The exchange of the expert-parallel layer on two gloo ranks on the CPU: count tables, split
sizes and row blocks (dummy rows that carry their origin) against the bookkeeping oracle."""
import os
import socket

import numpy as np
import torch
import torch.multiprocessing as mp

from oracle import r3_ep_oracle as EP


def _worker(rank, world, port, counts, out):
    import torch.distributed as dist
    from paper_2510_11370_b200 import ep          # loads the library; no GPU call is made here
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    el = counts.shape[1] // world
    send_counts = torch.from_numpy(counts[rank].reshape(world, el).astype(np.int32))
    recv_counts = ep.exchange_counts(send_counts)
    send_rows, recv_rows = ep.split_sizes(send_counts, recv_counts)
    # a row = (source rank, its position in the source's grouped order)
    n = int(counts[rank].sum())
    rows = torch.stack([torch.full((n,), rank, dtype=torch.int64), torch.arange(n)], dim=1)
    received = ep.exchange_rows(rows, send_rows, recv_rows)
    back = ep.exchange_rows(received, recv_rows, send_rows)
    out.put((rank, recv_counts.numpy().tolist(), send_rows, recv_rows, received.numpy().tolist(),
             bool(torch.equal(back, rows))))
    dist.destroy_process_group()


def test_two_ranks_exchange_counts_and_rows_as_the_oracle_says():
    world, E = 2, 8
    rng = np.random.default_rng(5)
    counts = rng.integers(0, 6, size=(world, E))
    counts[0, 5] = 0
    plans = EP.exchange_plan(counts)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, counts, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    el = E // world
    for rank, recv_counts, send_rows, recv_rows, received, round_trip in res:
        assert recv_counts == plans[rank]["recv_counts"]
        assert send_rows == plans[rank]["send_rows"] and recv_rows == plans[rank]["recv_rows"]
        # block from source s = the rows of s's grouped order that belong to this rank's experts
        want = []
        for s in range(world):
            first = int(counts[s, :rank * el].sum())
            want += [[s, first + i] for i in range(int(counts[s, rank * el:(rank + 1) * el].sum()))]
        assert received == want
        assert round_trip
