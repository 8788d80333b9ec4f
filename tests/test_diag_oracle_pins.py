"""Pins of the discrepancy-measure oracle (oracle/r3_diag_oracle.py) against things other than
itself: a hand-derived closed form (tests/golden/k3_and_etdf_closed_form.txt), analytic special
cases, invariants, and brute force with plain Python sets and loops."""
import math
import os

import numpy as np

from oracle import r3_diag_oracle as D

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "k3_and_etdf_closed_form.txt")


def golden():
    out = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        out[k] = [float(x) for x in v]
    return out


def test_k3_and_extreme_counts_match_the_hand_derived_values():
    g = golden()
    assert abs(D.kl_k3(g["p_train"], g["p_infer"]) - g["k3"][0]) < 1e-15
    assert D.extreme_counts(g["p_train"], g["p_infer"], g["taus"]).tolist() == [int(c) for c in g["counts"]]
    assert np.allclose(D.extreme_fraction(g["p_train"], g["p_infer"], g["taus"]),
                       np.array(g["counts"]) / 4)
    # ratios one part in a million either side of a threshold fall on the right side of it
    assert D.extreme_counts(g["near_p_train"], g["near_p_infer"], g["near_taus"]).tolist() == \
        [int(c) for c in g["near_counts"]]


def test_k3_special_cases():
    p = np.random.default_rng(0).random(1000) * 0.9 + 0.05
    assert D.kl_k3(p, p) == 0.0                                     # identical distributions
    c = 1.7                                                         # constant ratio: c - 1 - ln c
    assert abs(D.kl_k3(c * p / 2, p / 2) - (c - 1 - math.log(c))) < 1e-12
    q = np.random.default_rng(1).random(1000) * 0.9 + 0.05
    assert D.kl_k3(p, q) > 0                                        # r - 1 - ln r >= 0, = 0 iff r = 1
    # scalar loop with math.fsum
    ref = math.fsum(a / b - 1 - math.log(a / b) for a, b in zip(p, q)) / 1000
    assert abs(D.kl_k3(p, q) - ref) < 1e-13
    assert D.kl_k3([], []) == 0.0


def test_extreme_fraction_properties():
    rng = np.random.default_rng(2)
    p, q = rng.random(5000) * 0.9 + 0.05, rng.random(5000) * 0.9 + 0.05
    taus = [0.5, 1.0, 1.5, 2.0, 4.0, 1e9]
    f = D.extreme_fraction(p, q, taus)
    assert f[0] == 1.0 and f[-1] == 0.0                              # max(r, 1/r) >= 1 always
    assert np.all(np.diff(f) <= 0)                                   # non-increasing in tau
    assert np.array_equal(D.extreme_counts(p, q, taus), D.extreme_counts(q, p, taus))   # symmetric
    assert D.extreme_counts(p, p, [1.0])[0] == 0                     # strict inequality
    brute = [sum(1 for a, b in zip(p.tolist(), q.tolist()) if max(a / b, b / a) > t) for t in taus]
    assert D.extreme_counts(p, q, taus).tolist() == brute            # brute force, Python floats


def test_router_level_diff_against_sets_and_special_cases():
    rng = np.random.default_rng(3)
    L, T, E, K = 3, 40, 12, 4
    a = np.stack([np.stack([rng.permutation(E)[:K] for _ in range(T)]) for _ in range(L)])
    b = np.stack([np.stack([rng.permutation(E)[:K] for _ in range(T)]) for _ in range(L)])
    d = D.router_level_diff(a, b)
    assert d.shape == (L, T)
    for l in range(L):
        for t in range(T):
            assert d[l, t] == len(set(a[l, t]) - set(b[l, t])) == len(set(b[l, t]) - set(a[l, t]))
    assert np.all(D.router_level_diff(a, a) == 0)
    shuffled = a[:, :, ::-1]                                         # slot order does not matter
    assert np.all(D.router_level_diff(a, shuffled) == 0)
    disjoint = (a + K) % (2 * K + E)                                 # ids a..: make a disjoint record
    lo = np.tile(np.arange(K), (L, T, 1))
    hi = lo + K
    assert np.all(D.router_level_diff(lo, hi) == K)
    one = lo.copy()
    one[:, :, 0] = 2 * K                                             # exactly one choice replaced
    assert np.all(D.router_level_diff(lo, one) == 1)
    assert np.array_equal(D.router_level_diff(a, b), D.router_level_diff(b, a))
    h = D.router_level_histogram(d, K)
    assert h.sum() == L * T and h.shape == (K + 1,)
    assert all(h[v] == np.count_nonzero(d == v) for v in range(K + 1))
    del disjoint


def test_token_and_sequence_levels():
    d = np.array([[0, 2, 0, 1, 0],
                  [1, 0, 0, 3, 0],
                  [0, 4, 0, 0, 0]])                                  # L = 3 layers, T = 5 tokens
    choices, routers = D.token_level_diff(d)
    assert choices.tolist() == [1, 6, 0, 4, 0]
    assert routers.tolist() == [1, 2, 0, 2, 0]
    sums, means = D.sequence_level_diff(routers, [0, 2, 2, 5])       # lengths 2, 0, 3
    assert sums.tolist() == [3, 0, 2]
    assert np.allclose(means, [1.5, 0.0, 2 / 3])
    # at least one differing layer: the fraction the paper quotes per token
    assert np.count_nonzero(routers > 0) == 3
