"""Routing-record store (Section 4.2): pins of its oracle, and the host-side page pool of the
library against that oracle (no GPU needed: the pool is host code behind the C ABI)."""
import numpy as np
import pytest

from oracle import r3_store_oracle as S


def test_oracle_append_then_gather_is_concatenation_and_multi_turn_append_is_one_append():
    rng = np.random.default_rng(0)
    L, K, PT = 3, 4, 8
    pages = {p: np.full((L, PT, K), 255, dtype=np.uint8) for p in range(10)}
    rec_a = rng.integers(0, 200, size=(L, 19, K)).astype(np.uint8)
    rec_b = rng.integers(0, 200, size=(L, 5, K)).astype(np.uint8)
    ta, tb = [4, 1, 7], [9]
    n = S.append(pages, ta, 0, rec_a[:, :11], PT)          # turn 1
    n = S.append(pages, ta, n, rec_a[:, 11:], PT)          # turn 2 continues the same sequence
    assert n == 19
    S.append(pages, tb, 0, rec_b, PT)
    out = S.gather(pages, [ta, tb], [19, 5], PT, L, K, np.uint8)
    assert np.array_equal(out, np.concatenate([rec_a, rec_b], axis=1))
    # position p of a sequence sits in page table[p // PT] at offset p % PT, all layers together
    assert np.array_equal(pages[1][:, 3, :], rec_a[:, 11, :])
    # untouched slots keep their fill
    assert np.all(pages[7][:, 3:, :] == 255)


def test_oracle_shared_prefix_pages_give_identical_prefix_records():
    rng = np.random.default_rng(1)
    L, K, PT = 2, 2, 4
    pages = {p: np.zeros((L, PT, K), dtype=np.int16) for p in range(6)}
    prefix = rng.integers(0, 500, size=(L, 8, K)).astype(np.int16)
    tail1 = rng.integers(0, 500, size=(L, 3, K)).astype(np.int16)
    tail2 = rng.integers(0, 500, size=(L, 6, K)).astype(np.int16)
    S.append(pages, [0, 1, 2], 0, prefix, PT)
    S.append(pages, [0, 1, 2], 8, tail1, PT)
    S.append(pages, [0, 1, 3, 4], 8, tail2, PT)            # second sequence re-uses pages 0 and 1
    out = S.gather(pages, [[0, 1, 2], [0, 1, 3, 4]], [11, 14], PT, L, K, np.int16)
    assert np.array_equal(out[:, :8], prefix) and np.array_equal(out[:, 11:19], prefix)
    assert np.array_equal(out[:, 8:11], tail1) and np.array_equal(out[:, 19:], tail2)


def test_oracle_prefix_index():
    ix = S.PrefixIndex(6, 4)
    toks = list(range(100, 111))                           # 11 tokens: two full pages + 3
    assert ix.match(toks) == []
    t1 = ix.alloc(3)
    ix.publish(toks, t1)
    assert ix.match(toks) == t1[:2]                        # whole pages only
    assert ix.match(toks[:7]) == t1[:1]
    assert ix.match([1] + toks[1:]) == []                  # the first token differs: nothing
    assert ix.match(toks[:4] + [0, 0, 0, 0]) == t1[:1]
    # page t1[0] now has four users (its owner and three matches), t1[1] two, t1[2] one
    ix.release(t1)                                         # the owner goes: pages still used stay
    assert ix.match(toks[:4]) == t1[:1]
    for _ in range(4):
        ix.release(t1[:1])
    ix.release(t1[:2][1:])
    assert ix.match(toks) == []                            # last user gone: page left the index
    assert sorted(ix.free) == list(range(6))


# ---- the library's host-side pool against the oracle index --------------------------------------
@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import build
    build.build()
    from paper_2510_11370_b200 import r3 as mod
    return mod


def test_pagepool_follows_the_oracle_on_a_random_workload(r3):
    rng = np.random.default_rng(7)
    NP, PT = 64, 4
    pool, ix = r3.PagePool(NP, PT), S.PrefixIndex(NP, PT)
    live = []                                              # (tokens, pool table, oracle table)
    stems = [rng.integers(0, 50, size=rng.integers(4, 20)).tolist() for _ in range(5)]
    for step in range(400):
        if live and (rng.random() < 0.4 or pool.free_pages() < 8):
            toks, tp, to = live.pop(rng.integers(len(live)))
            pool.release(tp)
            ix.release(to)
        else:
            stem = stems[rng.integers(len(stems))]
            toks = stem[:rng.integers(1, len(stem) + 1)] + rng.integers(0, 50, size=rng.integers(0, 9)).tolist()
            mp, mo = pool.match(toks), ix.match(toks)
            assert len(mp) == len(mo)                      # same number of cached pages
            need = -(-len(toks) // PT) - len(mp)
            tp, to = mp + pool.alloc(need), mo + ix.alloc(need)
            pool.publish(toks, tp)
            ix.publish(toks, to)
            live.append((toks, tp, to))
        assert pool.free_pages() == len(ix.free)
        # pages shared between live sequences are shared identically on both sides
        for i, (ta, pa, oa) in enumerate(live):
            for tb, pb, ob in live[i + 1:]:
                assert [x == y for x, y in zip(pa, pb)] == [x == y for x, y in zip(oa, ob)]
    for toks, tp, to in live:
        pool.release(tp)
    assert pool.free_pages() == NP
    pool.close()


def test_pagepool_errors(r3):
    pool = r3.PagePool(4, 2)
    t = pool.alloc(4)
    with pytest.raises(r3.R3Error) as ei:
        pool.alloc(1)
    assert ei.value.code == 6                              # R3_ERR_OUT_OF_PAGES
    pool.release(t)
    with pytest.raises(r3.R3Error):
        pool.release([0])                                  # not in use
    with pytest.raises(r3.R3Error):
        pool.release([99])
    assert pool.free_pages() == 4
    with pytest.raises(ValueError):
        r3.PagePool(0, 4)
