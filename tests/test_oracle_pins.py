"""Pins for the CPU oracle: each function is checked against something other than itself -
closed forms, library routines on special cases, brute force over all M experts, finite
differences, and hand-derived values stored under tests/golden/."""
import itertools
import math
import os

import numpy as np
import pytest
import torch

from oracle import r3_oracle as O

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def tiny_layer(seed, T=6, d=5, E=4, F=3):
    r = rng(seed)
    x = r.standard_normal((T, d))
    w_r = r.standard_normal((E, d))
    wg = r.standard_normal((E, F, d)) * 0.7
    wu = r.standard_normal((E, F, d)) * 0.7
    wd = r.standard_normal((E, d, F)) * 0.7
    dy = r.standard_normal((T, d))
    return x, w_r, wg, wu, wd, dy


def load_golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.split("#")[0].strip()
            if line:
                rows.append([float(v) for v in line.split()])
    return rows


# ------------------------------------------------------------------ logits (first equation)
def test_logits_against_python_loops():
    r = rng(1)
    x = r.standard_normal((3, 4))
    w = r.standard_normal((5, 4))          # [E, d], non-square so a transposed operand fails
    s = O.router_logits(x, w)
    assert s.shape == (3, 5)
    for t in range(3):
        for i in range(5):
            ref = math.fsum(x[t, c] * w[i, c] for c in range(4))
            assert abs(s[t, i] - ref) < 1e-13


# ------------------------------------------------------------------ TopKMask
def test_topk_against_torch_topk_on_margin_safe_rows():
    r = rng(2)
    s = r.permuted(np.tile(np.arange(16.0), (40, 1)), axis=1)   # distinct values, margin 1
    for K in (1, 3, 16):
        got = O.topk_indices(s, K)
        ref = torch.topk(torch.from_numpy(s), K, dim=1).indices.numpy()
        assert np.array_equal(got, ref)


def test_topk_ties_go_to_lower_expert_and_order_is_descending():
    s = np.array([[1.0, 3.0, 3.0, 0.0, 3.0, 2.0],
                  [5.0, 5.0, 5.0, 5.0, 5.0, 5.0]])
    assert O.topk_indices(s, 2).tolist() == [[1, 2], [0, 1]]
    assert O.topk_indices(s, 4).tolist() == [[1, 2, 4, 5], [0, 1, 2, 3]]


def test_mask_has_exactly_K_ones():
    r = rng(3)
    s = r.standard_normal((20, 9))
    for K in range(1, 10):
        I = O.mask_from_indices(O.topk_indices(s, K), 9)
        assert np.all(I.sum(axis=1) == K) and set(np.unique(I)) <= {0.0, 1.0}


def test_record_validation_rejects_bad_records():
    with pytest.raises(ValueError):
        O.check_record(np.array([[0, 0]]), 4)
    with pytest.raises(ValueError):
        O.check_record(np.array([[0, 4]]), 4)
    with pytest.raises(ValueError):
        O.check_record(np.array([[-1, 2]]), 4)


# ------------------------------------------------------------------ gate (Eq. replay_gate)
def test_gate_closed_form_golden():
    # s = ln(1..6): exp(s_i) = i+1, so the gate over a set S is (i+1)/sum_{j in S}(j+1).
    for row in load_golden("replay_gate_closed_form.txt"):
        K = int(row[0])
        idx = np.array([[int(v) for v in row[1:1 + K]]])
        want = np.array(row[1 + K:1 + 2 * K])
        s = np.log(np.arange(1.0, 7.0))[None, :]
        got = O.replay_gate(s, idx)[0]
        assert np.allclose(got, want, rtol=0, atol=1e-15)


def test_gate_sums_to_one_positive_and_shift_invariant():
    r = rng(4)
    s = r.standard_normal((50, 12)) * 4
    idx = O.topk_indices(r.standard_normal((50, 12)), 5)      # arbitrary record
    g = O.replay_gate(s, idx)
    assert np.all(g > 0) and np.allclose(g.sum(axis=1), 1.0, atol=1e-12)
    g2 = O.replay_gate(s + 123.456, idx)
    assert np.allclose(g, g2, atol=1e-12)
    # extreme logits stay finite (stabilised softmax)
    g3 = O.replay_gate(s * 500, idx)
    assert np.all(np.isfinite(g3)) and np.allclose(g3.sum(axis=1), 1.0)


def test_gate_K1_is_one_and_KM_is_library_softmax():
    r = rng(5)
    s = r.standard_normal((30, 7))
    assert np.array_equal(O.replay_gate(s, O.topk_indices(s, 1)), np.ones((30, 1)))
    idx = np.tile(np.arange(7), (30, 1))
    ref = torch.softmax(torch.from_numpy(s), dim=1).numpy()
    assert np.allclose(O.replay_gate(s, idx), ref, atol=1e-14)


def test_gate_equals_full_softmax_renormalised_on_the_mask():
    r = rng(6)
    s = r.standard_normal((25, 10))
    idx = O.topk_indices(r.standard_normal((25, 10)), 4)
    p = torch.softmax(torch.from_numpy(s), dim=1).numpy()
    sel = np.take_along_axis(p, idx, axis=1)
    assert np.allclose(O.replay_gate(s, idx), sel / sel.sum(axis=1, keepdims=True), atol=1e-13)


def test_gate_slot_alignment_and_dense_form_agree():
    r = rng(7)
    s = r.standard_normal((15, 8))
    idx = np.stack([r.permutation(8)[:3] for _ in range(15)])   # arbitrary slot order
    g = O.replay_gate(s, idx)
    gd = O.gate_dense(s, O.mask_from_indices(idx, 8))
    assert np.allclose(np.take_along_axis(gd, idx, axis=1), g, atol=1e-14)
    off = np.ones_like(gd, dtype=bool)
    off[np.arange(15)[:, None], idx] = False
    assert np.all(gd[off] == 0)


# ------------------------------------------------------------------ experts
def test_expert_closed_form_scalar_golden():
    # d = F = 1: E(x) = wd * silu(wg x) * (wu x); values derived by hand in the golden file.
    for x, wg, wu, wd, want in load_golden("swiglu_scalar.txt"):
        got = O.swiglu_expert(np.array([[x]]), np.array([[wg]]), np.array([[wu]]),
                              np.array([[wd]]))
        assert abs(got[0, 0] - want) < 1e-12


def test_expert_against_library_formula_and_python_loops():
    r = rng(8)
    x = r.standard_normal((4, 5))
    wg, wu, wd = r.standard_normal((3, 5)), r.standard_normal((3, 5)), r.standard_normal((6, 3))
    got = O.swiglu_expert(x, wg, wu, wd)
    tx, tg, tu, td = map(torch.from_numpy, (x, wg, wu, wd))
    ref = (torch.nn.functional.silu(tx @ tg.T) * (tx @ tu.T)) @ td.T
    assert got.shape == (4, 6) and np.allclose(got, ref.numpy(), atol=1e-13)
    # scalar loops, no matmul at all
    for t in range(4):
        h = []
        for f in range(3):
            a = sum(wg[f, c] * x[t, c] for c in range(5))
            b = sum(wu[f, c] * x[t, c] for c in range(5))
            h.append(a / (1 + math.exp(-a)) * b)
        for c in range(6):
            assert abs(got[t, c] - sum(wd[c, f] * h[f] for f in range(3))) < 1e-12


def test_single_expert_layer_is_one_mlp_and_zero_down_gives_zero():
    x, w_r, wg, wu, wd, dy = tiny_layer(9, E=1)
    s = O.router_logits(x, w_r)
    y, g, _ = O.replay_output(x, s, np.zeros((6, 1), dtype=int), wg, wu, wd)
    assert np.allclose(y, O.swiglu_expert(x, wg[0], wu[0], wd[0]), atol=1e-14)
    x, w_r, wg, wu, wd, dy = tiny_layer(10)
    s = O.router_logits(x, w_r)
    y, _, _ = O.replay_output(x, s, O.topk_indices(s, 2), wg, wu, 0 * wd)
    assert np.all(y == 0)


# ------------------------------------------------------------------ output (Eq. replay_output)
def test_sparse_output_equals_sum_over_all_experts_brute_force():
    for seed, (T, d, E, F) in enumerate([(5, 4, 3, 2), (7, 6, 5, 4), (4, 8, 8, 6)]):
        x, w_r, wg, wu, wd, dy = tiny_layer(100 + seed, T, d, E, F)
        s = O.router_logits(x, w_r)
        r = rng(seed)
        for K in range(1, E + 1):
            idx = np.stack([r.permutation(E)[:K] for _ in range(T)])   # any record
            y, _, _ = O.replay_output(x, s, idx, wg, wu, wd)
            yd = O.replay_output_dense(x, s, O.mask_from_indices(idx, E), wg, wu, wd)
            assert np.allclose(y, yd, atol=1e-12)


def test_replay_with_own_topk_is_the_ordinary_layer():
    for seed in range(3):
        x, w_r, wg, wu, wd, dy = tiny_layer(200 + seed, T=9, d=6, E=6, F=4)
        s = O.router_logits(x, w_r)
        for K in (1, 2, 4, 6):
            y, _, _ = O.replay_output(x, s, O.topk_indices(s, K), wg, wu, wd)
            assert np.allclose(y, O.train_output(x, w_r, K, wg, wu, wd), atol=1e-12)


def test_replay_with_other_mask_differs_from_ordinary_layer():
    x, w_r, wg, wu, wd, dy = tiny_layer(210, T=9, d=6, E=6, F=4)
    s = O.router_logits(x, w_r)
    idx = O.topk_indices(-s, 2)                      # the two *least* likely experts
    y, _, _ = O.replay_output(x, s, idx, wg, wu, wd)
    assert not np.allclose(y, O.train_output(x, w_r, 2, wg, wu, wd))


def test_output_uses_slot_aligned_gates():
    # two experts with very different outputs and unequal gates: swapping gates must show
    x, w_r, wg, wu, wd, dy = tiny_layer(11, T=3, d=4, E=2, F=3)
    s = O.router_logits(x, w_r)
    idx = np.array([[1, 0]] * 3)
    y, g, eo = O.replay_output(x, s, idx, wg, wu, wd)
    for t in range(3):
        e1 = O.swiglu_expert(x[t:t + 1], wg[1], wu[1], wd[1])[0]
        e0 = O.swiglu_expert(x[t:t + 1], wg[0], wu[0], wd[0])[0]
        p = np.exp(s[t]) / np.exp(s[t]).sum()
        assert np.allclose(y[t], p[1] * e1 + p[0] * e0, atol=1e-13)
        assert np.allclose(eo[t, 0], e1) and np.allclose(eo[t, 1], e0)


def test_token_permutation_equivariance():
    x, w_r, wg, wu, wd, dy = tiny_layer(12, T=8)
    s = O.router_logits(x, w_r)
    idx = O.topk_indices(s + rng(0).standard_normal(s.shape), 2)
    out = O.layer_fwd_bwd(x, w_r, idx, wg, wu, wd, dy)
    p = rng(1).permutation(8)
    out2 = O.layer_fwd_bwd(x[p], w_r, idx[p], wg, wu, wd, dy[p])
    assert np.allclose(out["y"][p], out2["y"], atol=1e-13)
    assert np.allclose(out["ds"][p], out2["ds"], atol=1e-13)


# ------------------------------------------------------------------ permutation
def brute_permutation(idx, E):
    T, K = idx.shape
    rows = []
    for e in range(E):
        for t in range(T):
            for j in range(K):
                if idx[t, j] == e:
                    rows.append(t * K + j)
    return rows


def test_permutation_invariants_bruteforce_and_library_sort():
    r = rng(13)
    for T, E, K in [(1, 1, 1), (7, 5, 2), (33, 8, 3), (64, 16, 16), (100, 130, 4)]:
        idx = np.stack([r.permutation(E)[:K] for _ in range(T)])
        counts, offsets, ros, sor = O.permutation(idx, E)
        R = T * K
        assert counts.sum() == R and offsets[0] == 0 and offsets[-1] == R
        assert np.array_equal(offsets[1:] - offsets[:-1], counts)
        assert sorted(sor.tolist()) == list(range(R))
        assert np.array_equal(ros.reshape(-1)[sor], np.arange(R))
        keys = idx.reshape(-1)[sor]
        assert np.all(np.diff(keys) >= 0)
        tok = sor // K
        for e in range(E):
            seg = tok[offsets[e]:offsets[e + 1]]
            assert np.all(np.diff(seg) > 0)                       # stable: tokens ascending
        assert sor.tolist() == brute_permutation(idx, E)
        ref = torch.sort(torch.from_numpy(idx.reshape(-1)), stable=True).indices.numpy()
        assert np.array_equal(sor, ref)
        xs = r.standard_normal((T, 3))
        assert np.array_equal(O.permute_rows(xs, sor, K), xs[sor // K])


def test_permutation_with_empty_experts():
    idx = np.array([[3, 1], [1, 3], [3, 1]])
    counts, offsets, ros, sor = O.permutation(idx, 5)
    assert counts.tolist() == [0, 3, 0, 3, 0]
    assert offsets.tolist() == [0, 0, 3, 3, 6, 6]
    assert sor.tolist() == [1, 2, 5, 0, 3, 4]
    assert ros.tolist() == [[3, 0], [1, 4], [5, 2]]


# ------------------------------------------------------------------ gradient
def loss_of_logits(s, x, idx, wg, wu, wd, dy):
    y, _, _ = O.replay_output(x, s, idx, wg, wu, wd)
    return float(np.sum(dy * y))


def test_router_gradient_against_central_finite_differences():
    for seed, K in [(0, 1), (1, 2), (2, 3), (3, 4)]:
        x, w_r, wg, wu, wd, dy = tiny_layer(300 + seed, T=4, d=5, E=4, F=3)
        s = O.router_logits(x, w_r)
        r = rng(seed)
        idx = np.stack([r.permutation(4)[:K] for _ in range(4)])
        out = O.layer_fwd_bwd(x, w_r, idx, wg, wu, wd, dy)
        h = 1e-6
        fd = np.zeros_like(s)
        for t, i in itertools.product(range(4), range(4)):
            sp, sm = s.copy(), s.copy()
            sp[t, i] += h
            sm[t, i] -= h
            fd[t, i] = (loss_of_logits(sp, x, idx, wg, wu, wd, dy)
                        - loss_of_logits(sm, x, idx, wg, wu, wd, dy)) / (2 * h)
        scale = max(1.0, np.abs(fd).max())
        assert np.abs(out["ds"] - fd).max() / scale < 1e-6
        if K == 1:
            assert np.all(out["ds"] == 0)


def test_router_gradient_structure_and_autograd_second_opinion():
    x, w_r, wg, wu, wd, dy = tiny_layer(310, T=10, d=6, E=7, F=4)
    s = O.router_logits(x, w_r)
    idx = O.topk_indices(s + rng(5).standard_normal(s.shape), 3)
    out = O.layer_fwd_bwd(x, w_r, idx, wg, wu, wd, dy)
    ds = out["ds"]
    assert np.allclose(ds.sum(axis=1), 0, atol=1e-13)
    off = np.ones_like(ds, dtype=bool)
    off[np.arange(10)[:, None], idx] = False
    assert np.all(ds[off] == 0)
    # autograd through the dense printed form of the gate (mask is a constant)
    ts = torch.from_numpy(s).requires_grad_(True)
    I = torch.from_numpy(O.mask_from_indices(idx, 7))
    num = I * torch.exp(ts)
    g = num / num.sum(dim=1, keepdim=True)
    eo_dense = torch.stack([torch.from_numpy(O.swiglu_expert(x, wg[i], wu[i], wd[i]))
                            for i in range(7)], dim=1)            # [T, E, d]
    y = (g[:, :, None] * eo_dense).sum(dim=1)
    (y * torch.from_numpy(dy)).sum().backward()
    assert np.allclose(ds, ts.grad.numpy(), atol=1e-12)
    # dgates is the derivative of <dy, y> with respect to each gate
    assert np.allclose(out["dg"], np.einsum("td,tkd->tk", dy, out["eo"]))
    for t, j in [(0, 0), (3, 2), (9, 1)]:
        e = idx[t, j]
        assert abs(out["dg"][t, j] - float(dy[t] @ eo_dense[t, e].numpy())) < 1e-12


def test_per_token_evaluation_matches_batched():
    x, w_r, wg, wu, wd, dy = tiny_layer(320, T=12, d=6, E=6, F=4)
    s = O.router_logits(x, w_r)
    idx = O.topk_indices(s + rng(6).standard_normal(s.shape), 3)
    out = O.layer_fwd_bwd(x, w_r, idx, wg, wu, wd, dy)
    sel = [0, 5, 11]
    y, ds = O.layer_tokens(x[sel], w_r, idx[sel], wg, wu, wd, dy[sel])
    assert np.allclose(y, out["y"][sel], atol=1e-13)
    assert np.allclose(ds, out["ds"][sel], atol=1e-13)


def test_residual_stack_against_dense_definition_per_block():
    """Two residual blocks: every block's output is checked with the all-experts form of
    Eq. (replay_output) evaluated at that block's input, and x_L - x_0 is the sum of the outputs."""
    r = rng(500)
    T, d, E, F, K, L = 5, 4, 3, 3, 2, 3
    x0 = r.standard_normal((T, d))
    dy = r.standard_normal((T, d))
    layers, dense = [], []
    for l in range(L):
        _, w_r, wg, wu, wd, _ = tiny_layer(510 + l, T, d, E, F)
        idx = np.stack([r.permutation(E)[:K] for _ in range(T)])
        layers.append((w_r, idx, wg, wu, wd))
    xL, dss = O.replay_stack_tokens(x0, layers, dy)
    x = x0.copy()
    for l, (w_r, idx, wg, wu, wd) in enumerate(layers):
        s = O.router_logits(x, w_r)
        y = O.replay_output_dense(x, s, O.mask_from_indices(idx, E), wg, wu, wd)
        out = O.layer_fwd_bwd(x, w_r, idx, wg, wu, wd, dy)
        assert np.allclose(dss[l], out["ds"], atol=1e-13)
        x = x + y
    assert np.allclose(xL, x, atol=1e-12)
    # a subset of tokens followed on its own gives the same rows; `store` is applied per block
    sub = [1, 3]
    xs, _ = O.replay_stack_tokens(x0[sub], [(a, b[sub], c, e, f) for a, b, c, e, f in layers],
                                  dy[sub])
    assert np.allclose(xs, xL[sub], atol=1e-13)
    xr, _ = O.replay_stack_tokens(x0, layers, dy, store=lambda v: np.round(v, 2))
    assert np.array_equal(xr, np.round(xr, 2)) and not np.allclose(xr, xL, atol=1e-6)


# ------------------------------------------------------------------ planted mistakes are caught
def test_pins_catch_planted_mistakes(monkeypatch):
    """A wrong sign in silu, a transposed router weight or gates taken from the inference
    logits each break at least one of the checks above; spot-check three of them here."""
    x, w_r, wg, wu, wd, dy = tiny_layer(400, T=5, d=4, E=4, F=3)
    s = O.router_logits(x, w_r)
    idx = O.topk_indices(s, 2)
    good = O.replay_output(x, s, idx, wg, wu, wd)[0]
    monkeypatch.setattr(O, "silu", lambda z: z / (1.0 + np.exp(z)))
    bad = O.replay_output(x, s, idx, wg, wu, wd)[0]
    assert not np.allclose(good, bad)
    monkeypatch.undo()
    # gates from other logits change the output
    other = O.replay_output(x, s + rng(1).standard_normal(s.shape), idx, wg, wu, wd)[0]
    assert not np.allclose(good, other)


# ---------------------------------------------------------------------------------------------
# Update-stage backward to the layer input and the router weight
# ---------------------------------------------------------------------------------------------
def _tiny_layer(seed, T=5, d=6, E=4, K=2, F=5):
    rng = np.random.default_rng(seed)
    x = rng.normal(size=(T, d))
    w_r = rng.normal(size=(E, d)) * 0.5
    wg = rng.normal(size=(E, F, d)) * 0.4
    wu = rng.normal(size=(E, F, d)) * 0.4
    wd = rng.normal(size=(E, d, F)) * 0.4
    dy = rng.normal(size=(T, d))
    idx = np.stack([rng.permutation(E)[:K] for _ in range(T)])
    return x, w_r, idx, wg, wu, wd, dy


def _loss(x, w_r, idx, wg, wu, wd, dy):
    s = O.router_logits(x, w_r)
    y, _, _ = O.replay_output(x, s, idx, wg, wu, wd)
    return float(np.sum(dy * y))


def test_dsilu_is_the_derivative_of_silu():
    z = np.linspace(-6, 6, 41)
    h = 1e-6
    assert np.allclose(O.dsilu(z), (O.silu(z + h) - O.silu(z - h)) / (2 * h), atol=1e-8)


def test_input_gradient_matches_central_differences():
    x, w_r, idx, wg, wu, wd, dy = _tiny_layer(0)
    got = O.layer_bwd_input(x, w_r, idx, wg, wu, wd, dy)
    h = 1e-6
    num = np.zeros_like(x)
    for t in range(x.shape[0]):
        for c in range(x.shape[1]):
            xp, xm = x.copy(), x.copy()
            xp[t, c] += h
            xm[t, c] -= h
            num[t, c] = (_loss(xp, w_r, idx, wg, wu, wd, dy) - _loss(xm, w_r, idx, wg, wu, wd, dy)) / (2 * h)
    assert np.abs(got["dx"] - num).max() / np.abs(num).max() < 1e-7
    assert np.allclose(got["dx"], got["dx_expert"] + got["dx_router"])


def test_router_weight_gradient_matches_central_differences():
    x, w_r, idx, wg, wu, wd, dy = _tiny_layer(1)
    got = O.layer_bwd_input(x, w_r, idx, wg, wu, wd, dy)
    h = 1e-6
    num = np.zeros_like(w_r)
    for e in range(w_r.shape[0]):
        for c in range(w_r.shape[1]):
            wp, wm = w_r.copy(), w_r.copy()
            wp[e, c] += h
            wm[e, c] -= h
            num[e, c] = (_loss(x, wp, idx, wg, wu, wd, dy) - _loss(x, wm, idx, wg, wu, wd, dy)) / (2 * h)
    assert np.abs(got["dw_r"] - num).max() / np.abs(num).max() < 1e-7


def test_input_gradient_special_cases():
    x, w_r, idx, wg, wu, wd, dy = _tiny_layer(2, K=1)
    got = O.layer_bwd_input(x, w_r, idx, wg, wu, wd, dy)
    assert np.all(got["dx_router"] == 0) and np.all(got["dw_r"] == 0)   # K = 1: the gate is 1
    # and the expert path is then the gradient of one SwiGLU MLP per token (torch autograd, float64)
    xt = torch.tensor(x, requires_grad=True)
    out = torch.zeros(())
    for t in range(x.shape[0]):
        e = int(idx[t, 0])
        hmid = torch.nn.functional.silu(xt[t] @ torch.tensor(wg[e]).T) * (xt[t] @ torch.tensor(wu[e]).T)
        out = out + (torch.tensor(dy[t]) * (hmid @ torch.tensor(wd[e]).T)).sum()
    out.backward()
    assert np.allclose(got["dx"], xt.grad.numpy(), atol=1e-12)
    # zero upstream gradient -> zero gradients
    z = O.layer_bwd_input(x, w_r, idx, wg, wu, wd, np.zeros_like(dy))
    assert np.all(z["dx"] == 0) and np.all(z["dw_r"] == 0)


# ---------------------------------------------------------------------------------------------
# Update-stage backward to the expert weights
# ---------------------------------------------------------------------------------------------
@pytest.mark.parametrize("which", [0, 1, 2])
def test_expert_weight_gradients_match_central_differences(which):
    x, w_r, idx, wg, wu, wd, dy = _tiny_layer(10 + which, T=6, d=4, E=3, K=2, F=3)
    got = O.layer_bwd_weights(x, w_r, idx, wg, wu, wd, dy)
    ws = [wg, wu, wd]
    target = ws[which]
    h = 1e-6
    num = np.zeros_like(target)
    for pos in np.ndindex(*target.shape):
        keep = target[pos]
        target[pos] = keep + h
        up = _loss(x, w_r, idx, *ws, dy)
        target[pos] = keep - h
        dn = _loss(x, w_r, idx, *ws, dy)
        target[pos] = keep
        num[pos] = (up - dn) / (2 * h)
    mine = np.stack([got[e][which] for e in range(wg.shape[0])])
    assert np.abs(mine - num).max() / np.abs(num).max() < 1e-7


def test_expert_weight_gradients_autograd_second_opinion_and_special_cases():
    x, w_r, idx, wg, wu, wd, dy = _tiny_layer(20, T=7, d=5, E=4, K=2, F=3)
    idx[idx == 3] = 0                      # expert 3 is never recorded ...
    idx[:, 1] = np.where(idx[:, 0] == idx[:, 1], 1 + idx[:, 0] % 2, idx[:, 1])
    idx[idx == 3] = 2
    assert not np.any(idx == 3) and np.all(idx[:, 0] != idx[:, 1])
    got = O.layer_bwd_weights(x, w_r, idx, wg, wu, wd, dy)
    for m in got[3]:
        assert np.all(m == 0)              # ... so its weights get no gradient
    # torch autograd through the dense printed form (gate = masked softmax, constant mask)
    tw = [torch.tensor(w, requires_grad=True) for w in (wg, wu, wd)]
    xt = torch.tensor(x)
    s = xt @ torch.tensor(w_r).T
    mask = torch.zeros_like(s)
    mask.scatter_(1, torch.tensor(idx), 1.0)
    e = mask * torch.exp(s)
    gate = e / e.sum(dim=1, keepdim=True)
    y = torch.zeros_like(xt)
    for i in range(wg.shape[0]):
        o = (torch.nn.functional.silu(xt @ tw[0][i].T) * (xt @ tw[1][i].T)) @ tw[2][i].T
        y = y + gate[:, i:i + 1] * o
    (torch.tensor(dy) * y).sum().backward()
    for i in range(wg.shape[0]):
        for which in range(3):
            assert np.allclose(got[i][which], tw[which].grad[i].numpy(), atol=1e-12)
    # restricting the experts changes nothing for those computed; zero dy gives zero
    part = O.layer_bwd_weights(x, w_r, idx, wg, wu, wd, dy, experts=[1])
    assert list(part) == [1] and all(np.array_equal(a, b) for a, b in zip(part[1], got[1]))
    z = O.layer_bwd_weights(x, w_r, idx, wg, wu, wd, np.zeros_like(dy))
    assert all(np.all(m == 0) for i in z for m in z[i])


# ---------------------------------------------------------------------------------------------
# exact backward chain of a residual stack
# ---------------------------------------------------------------------------------------------
def _tiny_stack(seed, L=3, T=4, d=5, E=4, K=2, F=3):
    layers = []
    for l in range(L):
        x, w_r, idx, wg, wu, wd, dy = _tiny_layer(seed + l, T=T, d=d, E=E, K=K, F=F)
        layers.append((w_r, idx, wg * 0.7, wu * 0.7, wd * 0.7))
    x0, _, _, _, _, _, dy = _tiny_layer(seed + 100, T=T, d=d, E=E, K=K, F=F)
    return x0, layers, dy


def _stack_loss(x0, layers, dy):
    x = x0
    for (w_r, idx, wg, wu, wd) in layers:
        y, _, _ = O.replay_output(x, O.router_logits(x, w_r), idx, wg, wu, wd)
        x = x + y
    return float(np.sum(dy * x))


def test_stack_backward_chain_matches_central_differences():
    x0, layers, dy = _tiny_stack(40)
    got = O.replay_stack_bwd_tokens(x0, layers, dy)
    h = 1e-6
    num = np.zeros_like(x0)
    for pos in np.ndindex(*x0.shape):
        xp, xm = x0.copy(), x0.copy()
        xp[pos] += h
        xm[pos] -= h
        num[pos] = (_stack_loss(xp, layers, dy) - _stack_loss(xm, layers, dy)) / (2 * h)
    assert np.abs(got["dx0"] - num).max() / np.abs(num).max() < 1e-7
    # router weight of the middle block
    l = 1
    w_r = layers[l][0]
    numw = np.zeros_like(w_r)
    for pos in np.ndindex(*w_r.shape):
        keep = w_r[pos]
        w_r[pos] = keep + h
        up = _stack_loss(x0, layers, dy)
        w_r[pos] = keep - h
        dn = _stack_loss(x0, layers, dy)
        w_r[pos] = keep
        numw[pos] = (up - dn) / (2 * h)
    assert np.abs(got["dw_r"][l] - numw).max() / np.abs(numw).max() < 1e-6


def test_stack_backward_special_cases():
    x0, layers, dy = _tiny_stack(50)
    full = O.replay_stack_bwd_tokens(x0, layers, dy)
    # tokens are independent: a subset gives the same rows
    sel = np.array([0, 2])
    sub = O.replay_stack_bwd_tokens(x0[sel], [(w, i[sel], a, b, c) for (w, i, a, b, c) in layers],
                                    dy[sel])
    assert np.allclose(sub["dx0"], full["dx0"][sel], atol=1e-13)
    assert np.allclose(sub["ds"][0], full["ds"][0][sel], atol=1e-13)
    # one block: the chain is the layer's gradient plus the identity path
    one = O.replay_stack_bwd_tokens(x0, layers[:1], dy)
    w_r, idx, wg, wu, wd = layers[0]
    lay = O.layer_bwd_input(x0, w_r, idx, wg, wu, wd, dy)
    assert np.allclose(one["dx0"], dy + lay["dx"], atol=1e-13)
    # the last block's router gradient is that of the forward-only stack with the same dy
    xL, dss = O.replay_stack_tokens(x0, layers, dy)
    assert np.allclose(full["ds"][-1], dss[-1], atol=1e-13) and np.allclose(full["x_out"], xL)
    # zero experts (W_down = 0): every block is the identity, so dx0 = dy and ds = 0
    dead = [(w, i, a, b, np.zeros_like(c)) for (w, i, a, b, c) in layers]
    z = O.replay_stack_bwd_tokens(x0, dead, dy)
    assert np.array_equal(z["dx0"], dy) and all(np.all(s == 0) for s in z["ds"])


def test_stack_expert_weight_gradients_match_central_differences():
    """A weight of the FIRST block's experts reaches the loss through every later block."""
    x0, layers, dy = _tiny_stack(60, L=2, T=4, d=4, E=3, K=2, F=3)
    got = O.replay_stack_bwd_tokens(x0, layers, dy, expert_grads=True)
    h = 1e-6
    for which in range(3):
        target = layers[0][2 + which]
        num = np.zeros_like(target)
        for pos in np.ndindex(*target.shape):
            keep = target[pos]
            target[pos] = keep + h
            up = _stack_loss(x0, layers, dy)
            target[pos] = keep - h
            dn = _stack_loss(x0, layers, dy)
            target[pos] = keep
            num[pos] = (up - dn) / (2 * h)
        mine = np.stack([got["dw_experts"][0][e][which] for e in range(target.shape[0])])
        assert np.abs(mine - num).max() / np.abs(num).max() < 1e-6
