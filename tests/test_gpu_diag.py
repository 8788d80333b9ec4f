"""Discrepancy measures of Sections 3.1-3.2 on the GPU against the oracle: integer outputs bit for
bit, the k3 estimate within 1e-5 relative (terms formed in float32, summed in float64).  The
extreme-token counts are integer decisions that the kernel takes on float32 ratios and the oracle
on exact (float64) ones: they may differ only by tokens whose exact ratio lies within one float32
ulp of the threshold, and those tokens are counted."""
import numpy as np
import pytest
import torch

from oracle import r3_diag_oracle as D

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import r3 as mod
    return mod


def probs(n, seed, spread):
    """Per-token probabilities of two engines: p_infer uniform in (0.01, 1), p_train = p_infer
    times a log-normal ratio (a few extreme tokens, like the scatter of Figure 1)."""
    g = torch.Generator().manual_seed(seed)
    pi = torch.rand(n, generator=g) * 0.99 + 0.01
    ratio = torch.exp(torch.randn(n, generator=g) * spread)
    pt = (pi * ratio).clamp(1e-6, 1.0)
    return pt.float(), pi.float()


def check_extreme_counts(got, pt, pi, taus):
    """got[i] against the oracle's count for taus[i] (the float32 value the kernel is given).  A
    correctly rounded float32 ratio is within half an ulp of the exact one, so only a token whose
    exact ratio is within tau * 2^-23 of tau may be decided the other way."""
    big = D.extreme_ratio(pt, pi)
    near_total = 0
    for c, t in zip(got, taus):
        t = float(np.float32(t))
        lo = int(np.count_nonzero(big > t * (1 + 2.0 ** -23)))
        hi = int(np.count_nonzero(big > t * (1 - 2.0 ** -23)))
        near_total += hi - lo
        assert lo <= c <= hi, (t, c, lo, hi)
        if hi == lo:
            assert c == int(D.extreme_counts(pt, pi, [t])[0])
    return near_total


def test_extreme_counts_just_either_side_of_a_threshold(r3):
    """The hand-derived tokens of tests/golden/k3_and_etdf_closed_form.txt whose ratios sit one
    part in a million above and below tau = 2 (all values exact in float32)."""
    import os
    g = {}
    for line in open(os.path.join(os.path.dirname(__file__), "golden", "k3_and_etdf_closed_form.txt")):
        if line.strip() and not line.startswith("#"):
            k, *v = line.split()
            g[k] = [float(x) for x in v]
    pt = torch.tensor(g["near_p_train"], dtype=torch.float32)
    pi = torch.tensor(g["near_p_infer"], dtype=torch.float32)
    assert pt.double().tolist() == g["near_p_train"]             # stored exactly
    _, counts = r3.prob_discrepancy(pt.cuda(), pi.cuda(), g["near_taus"])
    assert counts.cpu().tolist() == [int(c) for c in g["near_counts"]]


@pytest.mark.parametrize("n,spread", [(1, 0.1), (1000, 0.05), (300_001, 0.3), (5_000_000, 0.1)])
def test_k3_and_extreme_counts(r3, n, spread):
    pt, pi = probs(n, n, spread)
    taus = [1.0, 1.05, 1.5, 2.0, 4.0, 10.0]
    kl, counts = r3.prob_discrepancy(pt.cuda(), pi.cuda(), taus)
    ref_kl = D.kl_k3(pt.numpy(), pi.numpy())
    # float32 terms (relative error below 1e-5 each), float64 sum
    assert abs(kl.item() - ref_kl) <= 1e-5 * abs(ref_kl) + 1e-12
    check_extreme_counts(counts.cpu().tolist(), pt.numpy(), pi.numpy(), taus)
    kl2, counts2 = r3.prob_discrepancy(pt.cuda(), pi.cuda(), taus)
    assert kl2.item() == kl.item() and torch.equal(counts, counts2)      # reproducible


def test_prob_discrepancy_edges(r3):
    kl, counts = r3.prob_discrepancy(torch.empty(0).cuda(), torch.empty(0).cuda(), [2.0])
    assert kl.item() == 0.0 and counts.item() == 0
    p = torch.full((777,), 0.3)
    kl, counts = r3.prob_discrepancy(p.cuda(), p.cuda(), [1.0, 0.5])
    assert kl.item() == 0.0 and counts.cpu().tolist() == [0, 777]
    with pytest.raises(r3.R3Error):
        r3.prob_discrepancy(p.cuda(), p.cuda(), list(range(1, 18)))      # more than 16 thresholds


def records(L, T, E, K, drift, seed, dtype):
    """Two records: b = a with each (layer, token) redrawn with probability `drift`."""
    rng = np.random.default_rng(seed)
    a = np.argsort(rng.random((L, T, E)), axis=2)[:, :, :K]
    b = np.argsort(rng.random((L, T, E)), axis=2)[:, :, :K]
    keep = rng.random((L, T, 1)) >= drift
    b = np.where(keep, np.take_along_axis(a, np.argsort(rng.random((L, T, K)), axis=2), axis=2), b)
    return torch.from_numpy(a.astype(np.int64)).to(dtype), torch.from_numpy(b.astype(np.int64)).to(dtype)


@pytest.mark.parametrize("L,T,E,K,dtype", [(1, 1, 4, 1, torch.uint8), (3, 300, 16, 4, torch.uint8),
                                           (48, 1000, 128, 8, torch.uint8),
                                           (2, 257, 300, 5, torch.int16)])
def test_record_diff_and_sequence_level(r3, L, T, E, K, dtype):
    a, b = records(L, T, E, K, 0.1, L * T, dtype)
    s = r3.make_shape(T, 8, E, K, 8, idx=dtype)
    diff, choices, routers, hist = r3.record_diff(s, L, a.cuda(), b.cuda())
    ref = D.router_level_diff(a.numpy(), b.numpy())
    assert np.array_equal(diff.cpu().numpy(), ref)
    rc, rr = D.token_level_diff(ref)
    assert np.array_equal(choices.cpu().numpy(), rc) and np.array_equal(routers.cpu().numpy(), rr)
    assert np.array_equal(hist.cpu().numpy(), D.router_level_histogram(ref, K))
    _, c2, r2, h2 = r3.record_diff(s, L, a.cuda(), b.cuda(), want_diff=False)
    assert torch.equal(c2, choices) and torch.equal(r2, routers) and torch.equal(h2, hist)
    # sequences of ragged lengths, one of them empty
    cuts = sorted(set([0, T // 3, T // 3, (2 * T) // 3, T]) | {0, T})
    cu = np.array([0] + [c for c in cuts if c > 0][:1] * 2 + cuts[2:] if T > 3 else [0, T], dtype=np.int32)
    cu = np.maximum.accumulate(cu)
    sums = r3.sequence_diff(routers, torch.from_numpy(cu).cuda())
    ref_sums, _ = D.sequence_level_diff(rr, cu)
    assert np.array_equal(sums.cpu().numpy(), ref_sums)
