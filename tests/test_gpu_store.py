"""Routing-record store on the GPU (r3_record_append / r3_record_gather, Section 4.2) against its
oracle, driven by the library's page pool: prefill, prefix hit, multi-turn append, ragged batch."""
import numpy as np
import pytest
import torch

from oracle import r3_store_oracle as S

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import r3 as mod
    return mod


def router_of_prefix(tokens, L, K, E, dtype):
    """Stand-in for the inference router: the record of position p depends only on the tokens up
    to p (and the layer), so equal prefixes give equal records - the property Section 4.2 uses."""
    out = np.zeros((L, len(tokens), K), dtype=dtype)
    h = 17
    for p, tok in enumerate(tokens):
        h = (h * 1000003 + tok + 1) % (2**31 - 1)
        for l in range(L):
            rng = np.random.default_rng(h + 7919 * l)
            out[l, p] = rng.permutation(E)[:K]
    return out


@pytest.mark.parametrize("L,K,E,PT,dtype", [(4, 8, 128, 16, torch.uint8), (2, 3, 40, 4, torch.uint8),
                                            (3, 8, 300, 8, torch.int16), (1, 1, 2, 1, torch.uint8)])
def test_store_round_trip_with_prefix_reuse_and_multi_turn(r3, L, K, E, PT, dtype):
    npdt = np.uint8 if dtype == torch.uint8 else np.int16
    rng = np.random.default_rng(L * 100 + K)
    NP, MAXP = 64, 16
    s = r3.make_shape(1, 8, E, K, 8, idx=dtype)
    page_bytes = r3.record_page_bytes(s, L, PT)
    pages = torch.zeros(NP * page_bytes, dtype=torch.uint8, device="cuda")
    o_pages = {p: np.zeros((L, PT, K), dtype=npdt) for p in range(NP)}
    pool = r3.PagePool(NP, PT)
    st = r3.new_status("cuda")

    stem = rng.integers(0, 1000, size=3 * PT + 1).tolist()
    seqs = [stem + rng.integers(0, 1000, size=n).tolist() for n in (5, 2 * PT, 0)]
    seqs.append(rng.integers(0, 1000, size=PT + 3).tolist())         # shares nothing
    tables, have = [], []

    def append_batch(which, new_counts):
        """One engine step: sequence i of `which` gets new_counts[i] more tokens recorded."""
        recs, pos0, cu = [], [], [0]
        for i, n_new in zip(which, new_counts):
            full = router_of_prefix(seqs[i][:have[i] + n_new], L, K, E, npdt)
            recs.append(full[:, have[i]:])
            pos0.append(have[i])
            cu.append(cu[-1] + n_new)
        rec = np.concatenate(recs, axis=1)
        bt = np.full((len(which), MAXP), -1, dtype=np.int32)
        for r, i in enumerate(which):
            bt[r, :len(tables[i])] = tables[i]
        r3.record_append(s, L, PT, pages, torch.from_numpy(bt).cuda(),
                         torch.tensor(pos0, dtype=torch.int32).cuda(),
                         torch.tensor(cu, dtype=torch.int32).cuda(),
                         torch.from_numpy(rec).to(dtype).cuda(), dev_status=st)
        for r, (i, n_new) in enumerate(zip(which, new_counts)):
            have[i] = S.append(o_pages, tables[i], have[i], recs[r], PT)

    # sequence 0: nothing cached; prefill in two steps, then publish
    for i, toks in enumerate(seqs):
        hit = pool.match(toks)
        need = -(-len(toks) // PT) - len(hit)
        tables.append(hit + pool.alloc(need))
        have.append(len(hit) * PT)                                    # cached tokens: not re-recorded
        if i == 0:
            assert hit == []
            append_batch([0], [PT + 2])
            append_batch([0], [len(toks) - have[0]])
        elif i in (1, 2):
            n_stem = len(stem) // PT                                  # the stem's full pages
            assert len(hit) == n_stem and hit == tables[0][:n_stem]
            if len(toks) > have[i]:
                append_batch([i], [len(toks) - have[i]])
        else:
            assert hit == []
            append_batch([i], [len(toks)])
        pool.publish(toks, tables[i])
    # a later turn: sequences 0 and 3 grow in the same step
    grow = [7, 2 * PT + 1]
    for i, g in zip((0, 3), grow):
        seqs[i] = seqs[i] + rng.integers(0, 1000, size=g).tolist()
        tables[i] += pool.alloc(-(-len(seqs[i]) // PT) - len(tables[i]))
    append_batch([0, 3], grow)
    assert st.item() == 0

    # training side: the packed record of the whole batch
    lens = [len(t) for t in seqs]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    bt = np.full((len(seqs), MAXP), -1, dtype=np.int32)
    for i, t in enumerate(tables):
        bt[i, :len(t)] = t
    out = r3.record_gather(s, L, PT, pages, torch.from_numpy(bt).cuda(),
                           torch.from_numpy(cu).cuda(), int(cu[-1]), dev_status=st)
    assert st.item() == 0
    ref = S.gather(o_pages, tables, lens, PT, L, K, npdt)
    assert np.array_equal(out.cpu().numpy(), ref)
    # and it is what the router would have produced for every sequence from scratch
    direct = np.concatenate([router_of_prefix(t, L, K, E, npdt) for t in seqs if len(t)], axis=1)
    assert np.array_equal(ref, direct)
    # device pages equal the oracle's pages byte for byte
    dev = pages.cpu().numpy().view(npdt).reshape(NP, L, PT, K)
    for p in range(NP):
        assert np.array_equal(dev[p], o_pages[p])
    pool.close()


def test_store_flags_positions_without_a_page(r3):
    L, K, PT = 2, 8, 4
    s = r3.make_shape(1, 8, 16, K, 8)
    pages = torch.zeros(4 * r3.record_page_bytes(s, L, PT), dtype=torch.uint8, device="cuda")
    st = r3.new_status("cuda")
    bt = torch.tensor([[0, -1]], dtype=torch.int32).cuda()
    rec = torch.ones((L, 6, K), dtype=torch.uint8).cuda()
    r3.record_append(s, L, PT, pages, bt, torch.zeros(1, dtype=torch.int32).cuda(),
                     torch.tensor([0, 6], dtype=torch.int32).cuda(), rec, dev_status=st)
    assert st.item() == r3.DEV_BAD_INDEX
    got = pages.cpu().numpy().reshape(4, L, PT, K)
    assert np.all(got[0] == 1) and np.all(got[1:] == 0)               # tokens 4, 5 were skipped
