"""Oracle of the expert-parallel exchange around the replayed layer.  TEST INFRASTRUCTURE ONLY:
imported by tests/ (never by the library or bench.py's product path).

The paper describes no parallelism; expert parallelism is this build's extension.  Nothing in
the mathematics changes: y_t of Eq. (replay_output) depends on token t and on the weights of its
K recorded experts alone, so the reference for the RESULT of an expert-parallel run is the plain
layer oracle on each rank's own tokens.  What needs an oracle of its own is the bookkeeping of
the exchange, written out here with Python loops:

  ranks r = 0..N-1, E experts, rank r owns the experts [r E/N, (r+1) E/N);
  every rank groups its (token, slot) rows by global expert (the layer's stable dispatch), so
  the rows bound for rank q are one contiguous block; after the exchange rank q holds, for every
  source rank s in order, that block: layout [source][local expert][row];
  the grouped expert GEMM wants [local expert][source][row].
"""
from __future__ import annotations

import numpy as np


def exchange_plan(counts_per_rank):
    """counts_per_rank [N][E]: rows of every global expert on every rank.  Returns for each
    rank q: send_rows [N] (rows it sends to each rank), recv_counts [N][E/N] (rows it receives
    from each source for each of its experts) and recv_rows [N]."""
    counts = np.asarray(counts_per_rank, dtype=np.int64)
    n, e = counts.shape
    assert e % n == 0
    el = e // n
    plans = []
    for q in range(n):
        send_rows = [int(counts[q, d * el:(d + 1) * el].sum()) for d in range(n)]
        recv_counts = [[int(counts[s, q * el + k]) for k in range(el)] for s in range(n)]
        recv_rows = [sum(row) for row in recv_counts]
        plans.append(dict(send_rows=send_rows, recv_counts=recv_counts, recv_rows=recv_rows))
    return plans


def regroup_map(recv_counts):
    """recv_counts [N][El].  Rows arrive as [source][expert][row]; returns (perm, offsets):
    perm[j] = arrival index of the row that stands at position j of the [expert][source][row]
    order, offsets [El+1] = first row of every local expert in that order."""
    rc = np.asarray(recv_counts, dtype=np.int64)
    n, el = rc.shape
    arrival_start = {}
    pos = 0
    for s in range(n):
        for k in range(el):
            arrival_start[(s, k)] = pos
            pos += int(rc[s, k])
    perm, offsets = [], [0]
    for k in range(el):
        for s in range(n):
            a = arrival_start[(s, k)]
            perm.extend(range(a, a + int(rc[s, k])))
        offsets.append(len(perm))
    return np.asarray(perm, dtype=np.int64), np.asarray(offsets, dtype=np.int64)


def regroup_rows(rows, recv_counts):
    """[source][expert][row] -> [expert][source][row]."""
    perm, offsets = regroup_map(recv_counts)
    return np.asarray(rows)[perm], offsets


def ungroup_rows(rows, recv_counts):
    """The inverse of regroup_rows."""
    perm, _ = regroup_map(recv_counts)
    out = np.empty_like(np.asarray(rows))
    out[perm] = rows
    return out


def dest_table(counts_all, me):
    """counts_all [N][E].  For rank `me`: dst_base[e] = row, in the owner's
    [local expert][source][row] buffer, of this rank's first row of expert e (rows of the owner's
    earlier experts from every source, then the rows of expert e from the sources before `me`);
    offsets_local [E/N + 1] = first row of each of `me`'s own experts in its buffer."""
    counts = np.asarray(counts_all, dtype=np.int64)
    n, e_total = counts.shape
    el = e_total // n
    dst_base = []
    for e in range(e_total):
        q, k = divmod(e, el)
        before = sum(int(counts[s, q * el + k2]) for k2 in range(k) for s in range(n))
        dst_base.append(before + sum(int(counts[s, e]) for s in range(me)))
    offsets_local = [0]
    for k in range(el):
        offsets_local.append(offsets_local[-1] + sum(int(counts[s, me * el + k]) for s in range(n)))
    return np.asarray(dst_base, dtype=np.int64), np.asarray(offsets_local, dtype=np.int64)
