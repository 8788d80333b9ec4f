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


# ---------------------------------------------------------------------------------------------
# The whole bookkeeping of one expert-parallel layer on two gloo ranks: ep.py's host functions
# carry the exchange, the oracles stand in for the library's kernels (dispatch, regrouping,
# destination table, experts, combine), and the result must be the plain layer oracle's on each
# rank's own tokens.
# ---------------------------------------------------------------------------------------------
def _tiny_layer(world):
    rng = np.random.default_rng(11)
    Tl, d, E, K, F = 37, 8, 8, 2, 8
    x = rng.standard_normal((world, Tl, d))
    dy = rng.standard_normal((world, Tl, d))
    w_r = rng.standard_normal((E, d)) * 0.3
    wg, wu = rng.standard_normal((E, F, d)) * 0.3, rng.standard_normal((E, F, d)) * 0.3
    wd = rng.standard_normal((E, d, F)) * 0.3
    idx = np.argsort(rng.random((world, Tl, E)), axis=2)[:, :, :K]
    idx[0][idx[0] == 5] = 4                                # expert 5 gets nothing from rank 0 ...
    for t in range(Tl):                                    # ... (keep the K experts distinct)
        if idx[0, t, 0] == idx[0, t, 1]:
            idx[0, t, 1] = 6
    return Tl, d, E, K, F, x, dy, w_r, wg, wu, wd, idx


def _layer_worker(rank, world, port, out):
    import torch.distributed as dist
    from oracle import r3_oracle as O
    from paper_2510_11370_b200 import ep
    os.environ.update(RANK=str(rank), WORLD_SIZE=str(world), MASTER_ADDR="127.0.0.1",
                      MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    Tl, d, E, K, F, x, dy, w_r, wg, wu, wd, idx = _tiny_layer(world)
    el = E // world
    xs, rec = x[rank], idx[rank]
    mine = slice(rank * el, (rank + 1) * el)

    # 1. dispatch (the library's r3_permute; here the oracle's stable grouping)
    counts, offsets, ros, sor = O.permutation(rec, E)
    xp = torch.from_numpy(xs[sor.astype(np.int64) // K])
    # 2. exchange of counts and rows (ep.py)
    send_counts = torch.from_numpy(counts.reshape(world, el).astype(np.int32))
    recv_counts = ep.exchange_counts(send_counts)
    send_rows, recv_rows = ep.split_sizes(send_counts, recv_counts)
    received = ep.exchange_rows(xp, send_rows, recv_rows)
    # 3. regroup to [expert][source][row] and run this rank's experts
    grouped, off_local = EP.regroup_rows(received.numpy(), recv_counts.numpy())
    outs = np.zeros_like(grouped)
    for k in range(el):
        lo, hi = int(off_local[k]), int(off_local[k + 1])
        if hi > lo:
            e = rank * el + k
            outs[lo:hi] = O.swiglu_expert(grouped[lo:hi], wg[e], wu[e], wd[e])
    # 4. way back
    back = EP.ungroup_rows(outs, recv_counts.numpy())
    returned = ep.exchange_rows(torch.from_numpy(back), recv_rows, send_rows).numpy()
    # 5. finish (the library's r3_replay_finish; here Eqs. replay_gate / replay_output)
    s = O.router_logits(xs, w_r)
    g = O.replay_gate(s, rec)
    eo = returned[ros.astype(np.int64)]                    # [Tl, K, d]
    y = np.einsum("tk,tkd->td", g, eo)
    ds = O.replay_gate_bwd(g, O.dgates(dy[rank], eo), rec, E)
    ref = O.layer_fwd_bwd(xs, w_r, rec, wg, wu, wd, dy[rank])
    ok_layer = bool(np.allclose(y, ref["y"], rtol=0, atol=1e-12) and
                    np.allclose(ds, ref["ds"], rtol=0, atol=1e-12))

    # ---- the direct-write form: all-gather of the counts, every rank's totals, destinations
    mine_counts = torch.from_numpy(counts.astype(np.int32))
    gathered = [torch.empty_like(mine_counts) for _ in range(world)]
    dist.all_gather(gathered, mine_counts)
    counts_all = torch.stack(gathered)
    totals = ep.owner_totals(counts_all, world)
    dst_base, off_direct = EP.dest_table(counts_all.numpy(), rank)
    # where each of this rank's grouped rows goes: (owner, row in the owner's buffer)
    owner = np.repeat(np.arange(E) // el, counts)
    place = np.concatenate([dst_base[e] + np.arange(counts[e]) for e in range(E)]).astype(np.int64)
    # the peer stores, emulated: everybody learns everybody's (owner, place, row)
    blob = [None] * world
    dist.all_gather_object(blob, (owner, place, xp.numpy()))
    buf = np.full((totals[rank], d), np.nan)
    for o_, p_, rows_ in blob:
        sel = o_ == rank
        buf[p_[sel]] = rows_[sel]
    same_buffer = bool(np.array_equal(buf, grouped) and
                       np.array_equal(off_direct, off_local))
    # the capacity check stops every rank together, or none
    raised = []
    for cap in (max(totals) - 1, max(totals)):
        try:
            ep.check_capacity(totals, cap)
            raised.append(False)
        except ValueError:
            raised.append(True)
    out.put((rank, ok_layer, same_buffer, totals, sum(recv_rows), raised))
    dist.destroy_process_group()


def test_two_ranks_whole_layer_bookkeeping_equals_the_layer_oracle():
    world = 2
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_layer_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    res = sorted(q.get(timeout=180) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    Tl, d, E, K = _tiny_layer(world)[:4]
    assert res[0][3] == res[1][3] and sum(res[0][3]) == world * Tl * K   # same totals everywhere
    for rank, ok_layer, same_buffer, totals, recv_total, raised in res:
        assert ok_layer                     # exchange + regroup + way back = the plain layer
        assert same_buffer                  # direct-write places = the regrouped all-to-all buffer
        assert totals[rank] == recv_total
        assert raised == [True, False]      # too small: every rank raises; large enough: none
