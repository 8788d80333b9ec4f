"""CPU oracle for the training/inference discrepancy measures of Sections 3.1 and 3.2.

TEST INFRASTRUCTURE ONLY (same rules as r3_oracle.py: imported by the tests, the smoke check and
the benchmark's reference legs, never by the product path, and sharing no code with it).

Plain numpy; floating point in float64, counts as Python / int64 integers.

  kl_k3            Eq. (kl), Section 3.1:  mean over tokens of  r - 1 - log r,  r = pi_train / pi_infer
  extreme_fraction Eq. (etdf), Section 3.1: F(tau) = fraction of tokens with max(r, 1/r) > tau
  router_level_diff, token_level_diff, sequence_level_diff
                   Section 3.2: numbers of differing expert choices between two routing records
                   (training and inference), per (layer, token), per token, per sequence.

Readings of Section 3.2 (the text gives no formulas): a record holds K distinct experts per
(layer, token); the number of differing expert choices of a router is K minus the size of the
intersection of the two K-sets (so 0 = same set, K = disjoint; the order of the slots does not
matter).  "Token-level": per token, the sum of these numbers over the layers, and the number of
layers whose router differs at all.  "Sequence-level": per sequence, the mean over its tokens
of the number of layers whose router differs ("the mean difference per token is approximately 6
routers").

Pins: tests/test_diag_oracle_pins.py.
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


# ----------------------------------------------------------------------------------------------
# Section 3.1
# ----------------------------------------------------------------------------------------------
def kl_k3(p_train, p_infer) -> float:
    """Eq. (kl): (1/|T|) sum_t [ r_t - 1 - log r_t ],  r_t = p_train[t] / p_infer[t]."""
    pt = np.asarray(p_train, dtype=F64).reshape(-1)
    pi = np.asarray(p_infer, dtype=F64).reshape(-1)
    if pt.size == 0:
        return 0.0
    r = pt / pi
    return float(np.sum(r - 1.0 - np.log(r)) / pt.size)


def extreme_ratio(p_train, p_infer) -> np.ndarray:
    """max(r_t, 1 / r_t) per token, r_t = p_train[t] / p_infer[t], in float64 (Eq. (etdf) is
    stated on real ratios; the stored probabilities are widened exactly)."""
    pt = np.asarray(p_train, dtype=F64).reshape(-1)
    pi = np.asarray(p_infer, dtype=F64).reshape(-1)
    return np.maximum(pt / pi, pi / pt)


def extreme_counts(p_train, p_infer, taus) -> np.ndarray:
    """Number of tokens with max(r, 1/r) > tau, one count per tau (Eq. (etdf) times |T|)."""
    big = extreme_ratio(p_train, p_infer)
    return np.array([int(np.count_nonzero(big > F64(t))) for t in taus], dtype=np.int64)


def extreme_fraction(p_train, p_infer, taus) -> np.ndarray:
    """Eq. (etdf): F(tau) for each tau."""
    n = np.asarray(p_train).size
    c = extreme_counts(p_train, p_infer, taus)
    return c.astype(F64) / max(n, 1)


# ----------------------------------------------------------------------------------------------
# Section 3.2
# ----------------------------------------------------------------------------------------------
def router_level_diff(rec_a, rec_b) -> np.ndarray:
    """rec_a, rec_b [L, T, K] expert ids.  Returns diff [L, T]: K - |set_a & set_b|."""
    a = np.asarray(rec_a, dtype=np.int64)
    b = np.asarray(rec_b, dtype=np.int64)
    assert a.shape == b.shape and a.ndim == 3
    L, T, K = a.shape
    out = np.empty((L, T), dtype=np.int64)
    for l in range(L):
        for t in range(T):
            out[l, t] = K - len(set(a[l, t].tolist()) & set(b[l, t].tolist()))
    return out


def router_level_histogram(diff, K: int) -> np.ndarray:
    """How many routers (layer, token) differ in 0, 1, ..., K expert choices."""
    return np.bincount(np.asarray(diff).reshape(-1), minlength=K + 1).astype(np.int64)


def token_level_diff(diff):
    """Per token: (sum over layers of the differing choices, number of layers that differ)."""
    d = np.asarray(diff)
    return d.sum(axis=0).astype(np.int64), (d > 0).sum(axis=0).astype(np.int64)


def sequence_level_diff(token_routers, cu_seqlens):
    """Per sequence s = tokens [cu[s], cu[s+1]): (sum of the tokens' differing-router counts,
    the mean per token)."""
    tr = np.asarray(token_routers, dtype=np.int64)
    cu = np.asarray(cu_seqlens, dtype=np.int64)
    sums = np.array([int(tr[cu[s]:cu[s + 1]].sum()) for s in range(len(cu) - 1)], dtype=np.int64)
    lens = np.diff(cu)
    means = np.where(lens > 0, sums / np.maximum(lens, 1), 0.0)
    return sums, means
