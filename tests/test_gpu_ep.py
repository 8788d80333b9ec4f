"""Expert parallelism on one GPU: the reordering kernels against the oracle, several ranks driven
in one process with the blocks carried between them by hand (the exchange itself is the only
step that is not run here), and one real process group of size one."""
import os
import socket

import numpy as np
import pytest
import torch

from oracle import r3_ep_oracle as EP
from oracle import r3_oracle as O
from paper_2510_11370_b200 import synth
from tests.helpers import f32, f64, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import r3 as mod
    return mod


@pytest.mark.parametrize("n_src,e_local,width", [(1, 4, 64), (2, 8, 136), (4, 3, 256), (8, 16, 64)])
def test_regroup_is_bit_exact_and_invertible(r3, n_src, e_local, width):
    rng = np.random.default_rng(n_src * 100 + e_local)
    rc = rng.integers(0, 40, size=(n_src, e_local))
    rc[rng.random(rc.shape) < 0.25] = 0
    rows = int(rc.sum())
    data = torch.randn(rows, width).to(torch.bfloat16)
    st = r3.new_status("cuda")
    perm, offsets = r3.ep_regroup_map(torch.from_numpy(rc.astype(np.int32)).cuda(), rows,
                                      dev_status=st)
    grouped = r3.ep_move_rows(data.cuda(), perm)
    back = r3.ep_move_rows(grouped, perm, inverse=True)
    torch.cuda.synchronize()
    assert st.item() == 0
    ref_perm, ref_off = EP.regroup_map(rc)
    assert np.array_equal(perm.cpu().numpy(), ref_perm)
    assert np.array_equal(offsets.cpu().numpy(), ref_off)
    assert torch.equal(grouped.cpu(), data[torch.from_numpy(ref_perm)])
    assert torch.equal(back.cpu(), data)


def test_regroup_rejects_a_table_that_does_not_add_up(r3):
    rc = torch.tensor([[3, 1], [0, 2]], dtype=torch.int32).cuda()
    st = r3.new_status("cuda")
    r3.ep_regroup_map(rc, 7, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() != 0


def _case(T_total, d, E, K, F):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name=f"ep{T_total}", T=T_total, d=d, E=E,
                     K=K, F=F)
    x, dy, w_r = synth.activations(w), synth.upstream_grad(w), synth.router_weight(w)
    wg, wu, wd = synth.expert_weights(w)
    s_ref = O.router_logits(f64(x), f64(w_r))
    idx = synth.make_record(w, torch.from_numpy(s_ref))
    return w, x, dy, w_r, wg, wu, wd, idx


@pytest.mark.parametrize("world", [2, 4])
def test_ranks_driven_by_hand_equal_the_single_gpu_layer(r3, world):
    """Tokens and experts split over `world` ranks; the all-to-alls are done by slicing.  Every
    rank's output must equal, bit for bit, the plain layer on the whole batch (same rows in the
    same order reach every expert), and the oracle within the bf16 bar."""
    from paper_2510_11370_b200.ep import EpRank
    T, d, E, K, F = 640, 256, 16, 4, 128
    w, x, dy, w_r, wg, wu, wd = _case(T, d, E, K, F)[:7]
    idx = _case(T, d, E, K, F)[7]
    dev = "cuda"
    xs, dys, idxs = x.to(dev), dy.to(dev), idx.to(dev)
    w_r_d, wg_d, wu_d, wd_d = w_r.to(dev), wg.to(dev), wu.to(dev), wd.to(dev)
    y_ref, ds_ref, g_ref = r3.replay_layer(r3.shape_of(w), xs, w_r_d, idxs, wg_d, wu_d, wd_d, dys)
    Tl, el = T // world, E // world
    ranks = [EpRank(q, world, Tl, d, E, K, F) for q in range(world)]
    tok = lambda q: slice(q * Tl, (q + 1) * Tl)
    send = [rk.dispatch(xs[tok(q)], w_r_d, idxs[tok(q)]) for q, rk in enumerate(ranks)]
    for q, rk in enumerate(ranks):                               # all-to-all of the counts
        rk.plan(torch.stack([send[s][q] for s in range(world)]))
    blocks = []                                                  # blocks[s][q]: rows s -> q
    for s, rk in enumerate(ranks):
        edges = np.concatenate([[0], np.cumsum(rk.send_rows)])
        blocks.append([rk.xp[edges[q]:edges[q + 1]] for q in range(world)])
    outs = []
    for q, rk in enumerate(ranks):                               # all-to-all of the rows
        received = torch.cat([blocks[s][q] for s in range(world)])
        assert [b.shape[0] for b in (blocks[s][q] for s in range(world))] == rk.recv_rows
        ex = slice(q * el, (q + 1) * el)
        outs.append(rk.experts(received, wg_d[ex].contiguous(), wu_d[ex].contiguous(),
                               wd_d[ex].contiguous()))
    for s, rk in enumerate(ranks):                               # the way back
        parts = []
        for q in range(world):
            edges = np.concatenate([[0], np.cumsum(ranks[q].recv_rows)])
            parts.append(outs[q][edges[s]:edges[s + 1]])
        y, dlogits, gates = rk.finish(torch.cat(parts), dys[tok(s)])
        torch.cuda.synchronize()
        assert rk.status.item() == 0
        assert torch.equal(y, y_ref[tok(s)]) and torch.equal(dlogits, ds_ref[tok(s)])
        assert torch.equal(gates, g_ref[tok(s)])
    ref = O.layer_fwd_bwd(f64(x), f64(w_r), idx.to(torch.int64).numpy(), f32(wg), f32(wu), f32(wd),
                          f64(dy))
    assert rel_err(f64(y_ref), ref["y"]) < 2e-2 and rel_err(f64(ds_ref), ref["ds"]) < 2e-2


def test_process_group_of_one_runs_the_real_collectives(r3):
    """ep_replay_layer with torch.distributed (NCCL, world size 1): the same calls a multi-GPU
    job makes; equal to the plain layer."""
    import torch.distributed as dist
    from paper_2510_11370_b200.ep import EpRank, ep_replay_layer
    T, d, E, K, F = 300, 256, 16, 4, 128
    w, x, dy, w_r, wg, wu, wd, idx = _case(T, d, E, K, F)
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    created = not dist.is_initialized()
    if created:
        os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        dist.init_process_group("nccl", rank=0, world_size=1)
    try:
        c = [t.cuda() for t in (x, w_r, idx, wg, wu, wd, dy)]
        y, dlogits, gates = ep_replay_layer(EpRank(0, 1, T, d, E, K, F), *c)
        y0, ds0, g0 = r3.replay_layer(r3.shape_of(w), *c)
        torch.cuda.synchronize()
        assert torch.equal(y, y0) and torch.equal(dlogits, ds0) and torch.equal(gates, g0)
    finally:
        if created:
            dist.destroy_process_group()


@pytest.mark.parametrize("n,E", [(1, 8), (2, 8), (4, 16), (8, 16)])
def test_destination_table_against_the_oracle(r3, n, E):
    rng = np.random.default_rng(n + E)
    counts = rng.integers(0, 50, size=(n, E))
    counts[rng.random(counts.shape) < 0.2] = 0
    dev_counts = torch.from_numpy(counts.astype(np.int32)).cuda()
    for me in range(n):
        dst_base, offsets_local = r3.ep_dest_table(dev_counts, me)
        ref_base, ref_off = EP.dest_table(counts, me)
        assert np.array_equal(dst_base.cpu().numpy(), ref_base)
        assert np.array_equal(offsets_local.cpu().numpy(), ref_off)


@pytest.mark.parametrize("world", [1, 2, 4])
def test_direct_write_ranks_equal_the_single_gpu_layer(r3, world):
    """The direct-write form with `world` ranks on one GPU: every rank's buffers live on this GPU,
    so "a peer's memory" is simply another tensor; the phases run rank after rank with the
    barriers of a real job replaced by program order.  Bit-identical to the plain layer."""
    from paper_2510_11370_b200.ep import EpDirectRank
    T, d, E, K, F = 640, 256, 16, 4, 128
    w, x, dy, w_r, wg, wu, wd, idx = _case(T, d, E, K, F)
    dev = "cuda"
    xs, dys, idxs = x.to(dev), dy.to(dev), idx.to(dev)
    w_r_d, wg_d, wu_d, wd_d = w_r.to(dev), wg.to(dev), wu.to(dev), wd.to(dev)
    y_ref, ds_ref, g_ref = r3.replay_layer(r3.shape_of(w), xs, w_r_d, idxs, wg_d, wu_d, wd_d, dys)
    Tl, el = T // world, E // world
    tok = lambda q: slice(q * Tl, (q + 1) * Tl)
    ranks = [EpDirectRank(q, world, Tl, d, E, K, F) for q in range(world)]
    counts_all = torch.stack([rk.route(xs[tok(q)], w_r_d, idxs[tok(q)])
                              for q, rk in enumerate(ranks)])           # the all-gather
    cap = max(max(rk.plan(counts_all) for rk in ranks), 1)               # one capacity for all
    assert all(rk.owner_rows == ranks[0].owner_rows for rk in ranks)
    recv = [torch.full((cap, d), float("nan"), dtype=torch.bfloat16, device=dev) for rk in ranks]
    outs = [torch.empty_like(b) for b in recv]
    for rk in ranks:
        rk.send([b.data_ptr() for b in recv], cap)
    torch.cuda.synchronize()                                             # barrier 1
    assert sum(rk.recv_rows for rk in ranks) == T * K
    for q, rk in enumerate(ranks):
        assert not torch.isnan(recv[q][:rk.recv_rows].float()).any()     # every row was written
        ex = slice(q * el, (q + 1) * el)
        rk.experts(recv[q], wg_d[ex].contiguous(), wu_d[ex].contiguous(), wd_d[ex].contiguous(),
                   outs[q])
    torch.cuda.synchronize()                                             # barrier 2
    for q, rk in enumerate(ranks):
        y, dlogits, gates = rk.finish([b.data_ptr() for b in outs], dys[tok(q)], cap)
        torch.cuda.synchronize()
        assert rk.status.item() == 0
        assert torch.equal(y, y_ref[tok(q)]) and torch.equal(dlogits, ds_ref[tok(q)])
        assert torch.equal(gates, g_ref[tok(q)])


def test_direct_form_refuses_buffers_that_are_too_small(r3):
    """A receive buffer smaller than the rows routed to its owner: the driver raises before any
    row is stored, and the kernels themselves never write beyond the capacity they are given (a
    canary behind the buffer stays intact, the status word reports the dropped rows)."""
    from paper_2510_11370_b200.ep import EpDirectRank, PeerBuffers, ep_replay_layer_direct
    T, d, E, K, F = 300, 256, 16, 4, 128
    w, x, dy, w_r, wg, wu, wd, idx = _case(T, d, E, K, F)
    c = [t.cuda() for t in (x, w_r, idx, wg, wu, wd, dy)]
    small = PeerBuffers.single(T * K - 100, d, torch.bfloat16, "cuda")
    with pytest.raises(ValueError, match="too small"):
        ep_replay_layer_direct(EpDirectRank(0, 1, T, d, E, K, F), small, *c)
    # the kernels alone, with the host check bypassed
    rk = EpDirectRank(0, 1, T, d, E, K, F)
    counts = rk.route(c[0], c[1], c[2])
    rk.plan(counts.view(1, -1))
    cap = T * K - 100
    buf = torch.zeros((T * K, d), dtype=torch.bfloat16, device="cuda")   # canary: rows >= cap
    rk.send([buf.data_ptr()], cap)
    torch.cuda.synchronize()
    assert rk.status.item() == r3.DEV_BAD_INDEX
    assert not buf[cap:].any() and buf[:cap].any()
    rk.status.zero_()
    row_ptr = r3.ep_slot_rows(rk.shape, 1, rk.idx, rk.row_of_slot, rk.offsets, rk.dst_base,
                              [buf.data_ptr()], cap, dev_status=rk.status)
    torch.cuda.synchronize()
    assert rk.status.item() == r3.DEV_BAD_INDEX
    beyond = (rk.row_of_slot.reshape(-1) >= cap)                         # one rank: place = row
    assert torch.all(row_ptr.reshape(-1)[beyond] == 0) and torch.all(row_ptr.reshape(-1)[~beyond] != 0)


def test_direct_form_driver_with_one_rank(r3):
    """ep_replay_layer_direct as a job of one rank (its own buffers), and, where this torch build
    can set it up for a group of one, with symmetric-memory buffers."""
    import torch.distributed as dist
    from paper_2510_11370_b200.ep import EpDirectRank, PeerBuffers, ep_replay_layer_direct
    T, d, E, K, F = 300, 256, 16, 4, 128
    w, x, dy, w_r, wg, wu, wd, idx = _case(T, d, E, K, F)
    c = [t.cuda() for t in (x, w_r, idx, wg, wu, wd, dy)]
    y0, ds0, g0 = r3.replay_layer(r3.shape_of(w), *c)
    bufs = PeerBuffers.single(T * K, d, torch.bfloat16, "cuda")
    y, dlogits, gates = ep_replay_layer_direct(EpDirectRank(0, 1, T, d, E, K, F), bufs, *c)
    torch.cuda.synchronize()
    assert torch.equal(y, y0) and torch.equal(dlogits, ds0) and torch.equal(gates, g0)
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    created = not dist.is_initialized()
    if created:
        os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        try:
            sym = PeerBuffers.symmetric(T * K, d, torch.bfloat16, torch.device("cuda", 0))
        except Exception as exc:                     # set-up of symmetric memory, not the library
            pytest.skip(f"symmetric memory unavailable for a group of one here: {exc!r}"[:200])
        y, dlogits, gates = ep_replay_layer_direct(EpDirectRank(0, 1, T, d, E, K, F), sym, *c)
        torch.cuda.synchronize()
        assert torch.equal(y, y0) and torch.equal(dlogits, ds0) and torch.equal(gates, g0)
    finally:
        if created:
            dist.destroy_process_group()
