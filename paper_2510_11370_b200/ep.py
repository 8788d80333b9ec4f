"""Expert parallelism around the replayed layer (an extension: the paper describes none).

N ranks, one process per GPU.  Router weights are replicated, the E experts are split: rank q owns
the experts [q E/N, (q+1) E/N).  Every rank routes its own tokens with the replayed record:

  1. dispatch   r3_permute with global expert numbers; rows for rank q are one contiguous block
  2. exchange   counts, then rows, with all-to-all (torch.distributed, NCCL over NVLink)
  3. experts    r3_ep_regroup_map / r3_ep_move_rows bring the received rows into
                [local expert][source][row]; r3_grouped_swiglu runs on them (T = rows, K = 1)
  4. return     rows go back through the inverse reordering and a second all-to-all
  5. finish     r3_replay_finish on the rank's own tokens (gate, combine, router-logit gradient)

Every step of the arithmetic runs in the library's kernels; this module only sequences them and
calls the collective.  The steps are methods of `EpRank` so that a test can drive several ranks
in one process and carry the blocks between them by hand; `ep_replay_layer` drives one rank with
real collectives.
"""
from __future__ import annotations

import torch
import torch.distributed as dist

from . import r3


def split_sizes(send_counts, recv_counts):
    """Rows this rank sends to / receives from every rank, from the two [N, E/N] count tables
    (one device-to-host copy when the tables live on a GPU)."""
    both = torch.stack([send_counts.sum(dim=1), recv_counts.sum(dim=1)]).cpu()
    return [int(v) for v in both[0]], [int(v) for v in both[1]]


def owner_totals(counts_all, world: int):
    """Rows every rank will RECEIVE in the direct-write form, from the all-gathered [N, E] count
    table (the same table on every rank, so every rank computes the same list): entry q is the
    number of rows routed to the experts of rank q by all ranks together.  One device-to-host copy
    when the table lives on a GPU."""
    n, e_total = counts_all.shape
    el = e_total // world
    totals = counts_all.reshape(n, world, el).sum(dim=(0, 2)).cpu()
    return [int(v) for v in totals]


def check_capacity(totals, capacity_rows: int):
    """Raises on EVERY rank (the totals are identical everywhere) when some owner's buffer cannot
    take the rows routed to it - before any rank has stored a row into a peer's memory."""
    worst = max(totals)
    if worst > capacity_rows:
        raise ValueError(f"receive buffers of {capacity_rows} rows are too small: rank "
                         f"{totals.index(worst)} is sent {worst} rows")


def exchange_counts(send_counts, group=None):
    """All-to-all of the [N, E/N] count table: row q goes to rank q; row s of the result is what
    rank s sends here."""
    recv_counts = torch.empty_like(send_counts)
    dist.all_to_all_single(recv_counts, send_counts, group=group)
    return recv_counts


def exchange_rows(rows, send_rows, recv_rows, group=None):
    """All-to-all of row blocks with the given split sizes."""
    received = torch.empty((sum(recv_rows),) + tuple(rows.shape[1:]), dtype=rows.dtype,
                           device=rows.device)
    dist.all_to_all_single(received, rows, output_split_sizes=recv_rows,
                           input_split_sizes=send_rows, group=group)
    return received


class EpRank:
    """One rank's state through one expert-parallel replayed layer."""

    def __init__(self, rank: int, world: int, T: int, d: int, E: int, K: int, F: int,
                 act=torch.bfloat16, router_w=torch.float32, idx_dtype=torch.uint8):
        if E % world:
            raise ValueError("the number of experts must be a multiple of the number of ranks")
        self.rank, self.world, self.e_local = rank, world, E // world
        self.shape = r3.make_shape(T, d, E, K, F, act=act, router=router_w, idx=idx_dtype)
        self.d, self.F, self.act = d, F, act
        self.status = None

    # -- 1: dispatch ---------------------------------------------------------------------------
    def dispatch(self, x, w_router, idx):
        """Returns send_counts [N, E/N] int32 (device): rows of each expert, by owner rank."""
        s = self.shape
        self.status = r3.new_status(x.device)
        self.idx = idx
        _, self.logits = r3.capture_topk_ws(s, 1, x, w_router, want_idx=False, want_logits=True)
        counts, _, self.row_of_slot, _, self.xp = r3.permute(s, idx, x, dev_status=self.status)
        self.send_counts = counts.view(self.world, self.e_local).contiguous()
        return self.send_counts

    # -- 2: sizes of the exchange (host) ---------------------------------------------------------
    def plan(self, recv_counts):
        """recv_counts [N, E/N] int32 (device): rows from each source for each local expert.
        Returns (send_rows, recv_rows), two lists of N ints (this synchronises with the GPU)."""
        self.recv_counts = recv_counts.contiguous()
        self.send_rows, self.recv_rows = split_sizes(self.send_counts, self.recv_counts)
        return self.send_rows, self.recv_rows

    # -- 3: experts on the received rows ---------------------------------------------------------
    def experts(self, received, w_gate, w_up, w_down):
        """received [sum(recv_rows), d] in [source][local expert][row] order; the weights are
        this rank's E/N experts.  Returns the expert outputs in the same order."""
        rows = received.shape[0]
        if rows == 0:
            return received.clone()
        perm, offsets = r3.ep_regroup_map(self.recv_counts, rows, dev_status=self.status)
        grouped = r3.ep_move_rows(received, perm)
        s_local = r3.make_shape(rows, self.d, self.e_local, 1, self.F, act=self.act)
        out = r3.grouped_swiglu(s_local, grouped, offsets, w_gate, w_up, w_down,
                                dev_status=self.status)
        return r3.ep_move_rows(out, perm, inverse=True)

    # -- 5: finish -------------------------------------------------------------------------------
    def finish(self, returned, dy):
        """returned [T K, d]: the expert outputs of this rank's rows, in its grouped order."""
        y, gates, dlogits = r3.replay_finish(self.shape, self.logits, self.idx, returned,
                                             self.row_of_slot, dy, dev_status=self.status)
        return y, dlogits, gates


class EpDirectRank:
    """One rank of the direct-write form: no collective carries rows.  After an all-gather of the
    per-expert counts every rank knows where each of its rows stands in its owner's
    [local expert][source][row] buffer, writes it there itself (r3_ep_dispatch_rows: plain stores
    into buffers this GPU can address - peers' memory over NVLink) and, once the owners have run
    their experts, pulls the outputs of its rows by address (r3_replay_finish_rows).  Two
    barriers of the job separate the phases; the receive and output buffers of all ranks must
    be addressable from every rank (peer access or symmetric memory)."""

    def __init__(self, rank: int, world: int, T: int, d: int, E: int, K: int, F: int,
                 act=torch.bfloat16, router_w=torch.float32, idx_dtype=torch.uint8):
        if E % world:
            raise ValueError("the number of experts must be a multiple of the number of ranks")
        self.rank, self.world, self.e_local = rank, world, E // world
        self.shape = r3.make_shape(T, d, E, K, F, act=act, router=router_w, idx=idx_dtype)
        self.d, self.F, self.E, self.act = d, F, E, act
        self.status = None

    def route(self, x, w_router, idx):
        """Logits and dispatch maps of this rank's tokens.  Returns counts [E] int32 (device)."""
        s = self.shape
        self.status = r3.new_status(x.device)
        self.x, self.idx = x, idx
        _, self.logits = r3.capture_topk_ws(s, 1, x, w_router, want_idx=False, want_logits=True)
        self.counts, self.offsets, self.row_of_slot, _, _ = r3.permute(s, idx,
                                                                       dev_status=self.status)
        return self.counts

    def plan(self, counts_all):
        """counts_all [N, E] (all-gathered).  Returns the rows this rank will receive; the rows
        every rank will receive are kept in `owner_rows` (identical on all ranks)."""
        self.dst_base, self.offsets_local = r3.ep_dest_table(counts_all.contiguous(), self.rank)
        self.owner_rows = owner_totals(counts_all, self.world)
        self.recv_rows = self.owner_rows[self.rank]
        return self.recv_rows

    def send(self, receive_buffers, capacity_rows: int):
        """receive_buffers: base addresses of every rank's [capacity_rows, d] receive buffer."""
        r3.ep_dispatch_rows(self.shape, self.world, self.x, self.idx, self.row_of_slot,
                            self.offsets, self.dst_base, receive_buffers, capacity_rows,
                            dev_status=self.status)

    def experts(self, received, w_gate, w_up, w_down, out):
        """This rank's experts on its receive buffer (already in expert-major order)."""
        if self.recv_rows:
            s_local = r3.make_shape(self.recv_rows, self.d, self.e_local, 1, self.F, act=self.act)
            r3.grouped_swiglu(s_local, received, self.offsets_local, w_gate, w_up, w_down, out,
                              dev_status=self.status)
        return out

    def finish(self, output_buffers, dy, capacity_rows: int):
        """output_buffers: base addresses of every rank's [capacity_rows, d] output buffer."""
        row_ptr = r3.ep_slot_rows(self.shape, self.world, self.idx, self.row_of_slot, self.offsets,
                                  self.dst_base, output_buffers, capacity_rows,
                                  dev_status=self.status)
        y, gates, dlogits = r3.replay_finish_rows(self.shape, self.logits, self.idx, row_ptr, dy,
                                                  dev_status=self.status)
        return y, dlogits, gates


class PeerBuffers:
    """The receive and output buffers of all ranks as seen from this rank: the rank's own two
    tensors, the base addresses of everybody's, and the job's barrier."""

    def __init__(self, received, outputs, receive_addresses, output_addresses, barrier):
        self.received, self.outputs = received, outputs
        self.capacity_rows = int(received.shape[0])      # the same on every rank
        self.receive_addresses, self.output_addresses = receive_addresses, output_addresses
        self.barrier = barrier

    @classmethod
    def single(cls, capacity_rows: int, d: int, dtype, device):
        """A job of one rank: the rank's own memory, no barrier needed beyond stream order."""
        rec = torch.empty((max(capacity_rows, 1), d), dtype=dtype, device=device)
        out = torch.empty_like(rec)
        return cls(rec, out, [rec.data_ptr()], [out.data_ptr()], lambda: None)

    @classmethod
    def symmetric(cls, capacity_rows: int, d: int, dtype, device, group=None):
        """Buffers of the same size on every rank, mapped into every rank's address space
        (torch symmetric memory: NVLink peer mappings).  capacity_rows must cover the worst case
        this job can route to one rank (at most world x T x K)."""
        import torch.distributed._symmetric_memory as symm
        group = group if group is not None else dist.group.WORLD
        rec = symm.empty((max(capacity_rows, 1), d), dtype=dtype, device=device)
        out = symm.empty((max(capacity_rows, 1), d), dtype=dtype, device=device)
        h_rec = symm.rendezvous(rec, group=group)
        h_out = symm.rendezvous(out, group=group)

        def barrier():
            torch.cuda.current_stream().synchronize()
            dist.barrier(group=group)

        return cls(rec, out, list(h_rec.buffer_ptrs), list(h_out.buffer_ptrs), barrier)


def ep_replay_layer_direct(state: "EpDirectRank", buffers: PeerBuffers, x, w_router, idx, w_gate,
                           w_up, w_down, dy, group=None):
    """One expert-parallel replayed layer in the direct-write form: (y, dlogits, gates).  The only
    collective is the all-gather of the [E] row counts."""
    counts = state.route(x, w_router, idx)
    if state.world > 1:
        counts_all = torch.empty((state.world, state.E), dtype=counts.dtype, device=counts.device)
        dist.all_gather_into_tensor(counts_all, counts, group=group)
    else:
        counts_all = counts.view(1, -1)
    state.plan(counts_all)
    # every rank sees the same totals: all of them stop here together, before anybody has
    # written into a peer's memory (the kernels also refuse to store beyond the capacity)
    check_capacity(state.owner_rows, buffers.capacity_rows)
    state.send(buffers.receive_addresses, buffers.capacity_rows)
    buffers.barrier()                       # every rank's rows have landed everywhere
    state.experts(buffers.received, w_gate, w_up, w_down, buffers.outputs)
    buffers.barrier()                       # every owner's outputs are complete
    result = state.finish(buffers.output_addresses, dy, buffers.capacity_rows)
    buffers.barrier()                       # nobody overwrites a buffer that is still being read
    return result


def ep_replay_layer(state: EpRank, x, w_router, idx, w_gate, w_up, w_down, dy, group=None):
    """One expert-parallel replayed layer on this rank with torch.distributed collectives:
    (y [T,d], dlogits [T,E], gates [T,K]).  w_gate / w_up / w_down hold this rank's experts."""
    send_counts = state.dispatch(x, w_router, idx)
    send_rows, recv_rows = state.plan(exchange_counts(send_counts, group))
    received = exchange_rows(state.xp, send_rows, recv_rows, group)
    out = state.experts(received, w_gate, w_up, w_down)
    returned = exchange_rows(out, recv_rows, send_rows, group)
    return state.finish(returned, dy)
