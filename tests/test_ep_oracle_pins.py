"""Pins of the expert-parallel bookkeeping oracle: conservation of rows, the exchange seen from
both ends, and the regrouping against a sort by (expert, source) keys."""
import numpy as np

from oracle import r3_ep_oracle as EP


def _counts(seed, n, e):
    rng = np.random.default_rng(seed)
    c = rng.integers(0, 7, size=(n, e))
    c[rng.random((n, e)) < 0.2] = 0
    return c


def test_exchange_plan_conserves_rows_and_matches_at_both_ends():
    for n, e in [(1, 4), (2, 8), (4, 16)]:
        counts = _counts(n * 10 + e, n, e)
        plans = EP.exchange_plan(counts)
        for q in range(n):
            assert sum(plans[q]["send_rows"]) == counts[q].sum()
            for s in range(n):
                # what q expects from s is what s sends to q
                assert plans[q]["recv_rows"][s] == plans[s]["send_rows"][q]
        total_recv = sum(sum(p["recv_rows"]) for p in plans)
        assert total_recv == counts.sum()


def test_regroup_equals_a_stable_sort_by_expert_then_source():
    rc = _counts(3, 3, 5)
    src_of, exp_of = [], []
    for s in range(rc.shape[0]):
        for k in range(rc.shape[1]):
            src_of += [s] * int(rc[s, k])
            exp_of += [k] * int(rc[s, k])
    src_of, exp_of = np.array(src_of), np.array(exp_of)
    rows = np.arange(len(src_of))[:, None] * np.ones((1, 3))
    got, offsets = EP.regroup_rows(rows, rc)
    order = np.lexsort((np.arange(len(src_of)), src_of, exp_of))     # expert, then source, stable
    assert np.array_equal(got[:, 0], order)
    assert np.array_equal(offsets, np.concatenate([[0], np.cumsum(rc.sum(axis=0))]))
    assert np.array_equal(EP.ungroup_rows(got, rc), rows)


def test_regroup_special_cases():
    # one source: nothing moves
    rc = np.array([[2, 0, 3]])
    rows = np.arange(5)[:, None]
    got, offsets = EP.regroup_rows(rows, rc)
    assert np.array_equal(got, rows) and list(offsets) == [0, 2, 2, 5]
    # one local expert: nothing moves either
    rc = np.array([[2], [0], [4]])
    rows = np.arange(6)[:, None]
    assert np.array_equal(EP.regroup_rows(rows, rc)[0], rows)
    # no rows at all
    got, offsets = EP.regroup_rows(np.zeros((0, 2)), np.zeros((2, 3), dtype=int))
    assert got.shape == (0, 2) and list(offsets) == [0, 0, 0, 0]


def test_dest_table_agrees_with_the_regrouped_order():
    """Writing every source's block straight to dst_base must give the buffer that exchanging
    and regrouping gives."""
    n, e_total = 3, 6
    counts = _counts(9, n, e_total)
    el = e_total // n
    for q in range(n):                                   # owner
        rc = np.array([[counts[s, q * el + k] for k in range(el)] for s in range(n)])
        # rows tagged (source, expert, i), in arrival order [source][expert][row]
        tags = [(s, k, i) for s in range(n) for k in range(el) for i in range(rc[s, k])]
        regrouped, offsets = EP.regroup_rows(np.array(tags).reshape(-1, 3), rc)
        direct = np.full((len(tags), 3), -1)
        for s in range(n):                               # every source writes its own rows
            dst_base, _ = EP.dest_table(counts, s)
            for k in range(el):
                for i in range(rc[s, k]):
                    direct[dst_base[q * el + k] + i] = (s, k, i)
        assert np.array_equal(direct, regrouped)
        assert np.array_equal(EP.dest_table(counts, q)[1], offsets)
