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


def ep_replay_layer(state: EpRank, x, w_router, idx, w_gate, w_up, w_down, dy, group=None):
    """One expert-parallel replayed layer on this rank with torch.distributed collectives:
    (y [T,d], dlogits [T,E], gates [T,K]).  w_gate / w_up / w_down hold this rank's experts."""
    send_counts = state.dispatch(x, w_router, idx)
    send_rows, recv_rows = state.plan(exchange_counts(send_counts, group))
    received = exchange_rows(state.xp, send_rows, recv_rows, group)
    out = state.experts(received, w_gate, w_up, w_down)
    returned = exchange_rows(out, recv_rows, send_rows, group)
    return state.finish(returned, dy)
