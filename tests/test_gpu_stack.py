"""A stack of residual MoE blocks with replayed routing (benchmark configuration 5) through the
C ABI against the oracle.  Every block's record is an input: it is drawn from the logits of the
stack's INPUT activations under that block's router (plus drift noise), so it does not depend on
computed state and the same record goes to both sides."""
import numpy as np
import pytest
import torch

from oracle import r3_oracle as O
from paper_2510_11370_b200 import synth
from tests.helpers import f64, rel_err

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import r3 as mod
    return mod


def bf16_store(v):
    return torch.from_numpy(np.ascontiguousarray(v)).to(torch.bfloat16).to(torch.float64).numpy()


def f32_store(v):
    return v.astype(np.float32).astype(np.float64)


class LayerExperts:
    """float64 view of the experts of one layer of a stacked [L, E, ...] device tensor."""

    def __init__(self, t, l):
        self.t, self.l = t, l

    def __len__(self):
        return self.t.shape[1]

    def __getitem__(self, i):
        return self.t[self.l, int(i)].to(torch.float64).cpu().numpy()


def build_stack(w, L, dev="cuda"):
    """Stacked per-layer tensors on the device, x0/dy, and per-layer records made from the
    oracle's logits of x0."""
    x0 = synth.activations(w, dev)
    dy = synth.upstream_grad(w, dev)
    w_r = torch.stack([synth.router_weight(w, dev, l) for l in range(L)])
    wg = torch.empty((L, w.E, w.F, w.d), dtype=w.act_dtype, device=dev)
    wu = torch.empty((L, w.E, w.F, w.d), dtype=w.act_dtype, device=dev)
    wd = torch.empty((L, w.E, w.d, w.F), dtype=w.act_dtype, device=dev)
    for l in range(L):
        a, b, c = synth.expert_weights(w, dev, l)
        wg[l], wu[l], wd[l] = a, b, c
        del a, b, c
    x0_64 = f64(x0)
    recs = []
    for l in range(L):
        s0 = O.router_logits(x0_64, f64(w_r[l]))
        recs.append(synth.make_record(w, torch.from_numpy(s0), l))
    idx = torch.stack(recs).to(dev)
    return x0, dy, w_r, wg, wu, wd, idx


def check_stack(r3, w, L, sel, tol, store, ds_layers=None):
    x0, dy, w_r, wg, wu, wd, idx = build_stack(w, L)
    s = r3.shape_of(w)
    st = r3.new_status("cuda")
    x_out, dlogits = r3.replay_stack(s, L, x0, w_r, idx, wg, wu, wd, dy, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    idx_np = idx.cpu().to(torch.int64).numpy()
    layers = [(f64(w_r[l]), idx_np[l][sel], LayerExperts(wg, l), LayerExperts(wu, l),
               LayerExperts(wd, l)) for l in range(L)]
    x_ref, ds_ref = O.replay_stack_tokens(f64(x0)[sel], layers, f64(dy)[sel], store=store)
    x_got = f64(x_out)[sel]
    err_x = np.abs(x_got - x_ref).max() / np.abs(x_ref).max()
    # Per-block quantities keep the per-layer bar `tol`.  The stack output passes through L
    # storage roundings of the running sum: an error in y_l that straddles a rounding boundary
    # moves an element by one ulp of the stored type (2^-8 relative for bf16, 2^-23 for f32), and
    # these moves add up like a random walk over the L blocks.
    ulp = 2.0 ** -8 if w.act == "bf16" else 2.0 ** -23
    tol_x = tol + np.sqrt(L) * ulp
    assert err_x < tol_x, err_x
    errs = []
    for l in range(L if ds_layers is None else ds_layers):
        got = dlogits[l].cpu().numpy().astype(np.float64)[sel]
        errs.append(np.abs(got - ds_ref[l]).max() / np.abs(ds_ref[l]).max())
    worst = max(errs)
    assert worst < tol, [round(float(e), 4) for e in errs]
    # a second run is bitwise identical
    x2, dl2 = r3.replay_stack(s, L, x0, w_r, idx, wg, wu, wd, dy)
    assert torch.equal(x_out, x2) and torch.equal(dlogits, dl2)
    print(f"{w.name} x{L}: x_L err {err_x:.2e} (bound {tol_x:.2e}), worst block dlogits err "
          f"{worst:.2e} (bound {tol:.0e})")
    return err_x, worst


def test_small_stack_fp32_all_tokens(r3):
    w = synth.scaled(synth.WORKLOADS["c1_tiny_fp32"], name="stack_f32", T=100, d=64, E=8, K=2,
                     F=64, record="noise", sigma=0.3)
    check_stack(r3, w, 4, np.arange(100), 1e-5, f32_store)


def test_small_stack_bf16_all_tokens(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="stack_bf16", T=300, d=256, E=16,
                     K=4, F=128)
    check_stack(r3, w, 3, np.arange(300), 2e-2, bf16_store)


def test_one_block_stack_is_layer_plus_residual(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="stack1", T=200, d=256, E=16, K=4,
                     F=128)
    x0, dy, w_r, wg, wu, wd, idx = build_stack(w, 1)
    s = r3.shape_of(w)
    x1, dl = r3.replay_stack(s, 1, x0, w_r, idx, wg, wu, wd, dy)
    y, ds, _ = r3.replay_layer(s, x0, w_r[0], idx[0], wg[0], wu[0], wd[0], dy)
    assert torch.equal(dl[0], ds)
    assert (x1.float() - (x0.float() + y.float())).abs().max().item() <= 0.0625   # <= 1 bf16 ulp


def build_blocks(w, L, dev="cuda"):
    """Independent blocks: per-layer inputs x_l, dy_l, weights, and records from the oracle's
    logits of each x_l."""
    x = torch.stack([synth.activations(w, dev, l) for l in range(L)])
    dy = torch.stack([synth.upstream_grad(w, dev, l) for l in range(L)])
    w_r = torch.stack([synth.router_weight(w, dev, l) for l in range(L)])
    wg = torch.empty((L, w.E, w.F, w.d), dtype=w.act_dtype, device=dev)
    wu = torch.empty((L, w.E, w.F, w.d), dtype=w.act_dtype, device=dev)
    wd = torch.empty((L, w.E, w.d, w.F), dtype=w.act_dtype, device=dev)
    recs = []
    for l in range(L):
        a, b, c = synth.expert_weights(w, dev, l)
        wg[l], wu[l], wd[l] = a, b, c
        del a, b, c
        s_l = O.router_logits(f64(x[l]), f64(w_r[l]))
        recs.append(synth.make_record(w, torch.from_numpy(s_l), l))
    return x, dy, w_r, wg, wu, wd, torch.stack(recs).to(dev)


def check_blocks(r3, w, L, n_samples, tol, rows_of_blocks=()):
    x, dy, w_r, wg, wu, wd, idx = build_blocks(w, L)
    s = r3.shape_of(w)
    st = r3.new_status("cuda")
    y, dlogits = r3.replay_blocks(s, L, x, w_r, idx, wg, wu, wd, dy, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    rng = np.random.default_rng(w.T + L)
    worst_y = worst_ds = 0.0
    for l in range(L):
        # the sampled tokens of block l through the oracle's layer as a batch of their own
        sel = np.sort(rng.choice(w.T, size=min(n_samples, w.T), replace=False))
        tsel = torch.from_numpy(sel).to(x.device)
        rec = idx[l][tsel].cpu().to(torch.int64).numpy()
        ref = O.layer_fwd_bwd(f64(x[l][tsel]), f64(w_r[l]), rec, LayerExperts(wg, l),
                              LayerExperts(wu, l), LayerExperts(wd, l), f64(dy[l][tsel]))
        worst_y = max(worst_y, rel_err(f64(y[l][tsel]), ref["y"]))
        worst_ds = max(worst_ds, rel_err(f64(dlogits[l][tsel]), ref["ds"]))
    assert worst_y < tol and worst_ds < tol, (worst_y, worst_ds)
    # block l of the batch equals r3_replay_layer on its own
    l = L - 1
    y1, ds1, _ = r3.replay_layer(s, x[l], w_r[l], idx[l], wg[l], wu[l], wd[l], dy[l])
    assert torch.equal(y1, y[l]) and torch.equal(ds1, dlogits[l])
    # all rows of chosen experts of chosen blocks: the dispatch and the grouped GEMM output o
    worst_o = 0.0
    for l in rows_of_blocks:
        rec = idx[l].cpu().to(torch.int64).numpy()
        counts, offsets, ros, sor = O.permutation(rec, w.E)
        got = r3.permute(s, idx[l], x[l], dev_status=st)
        for a, b in zip(got[:4], (counts, offsets, ros, sor)):
            assert np.array_equal(a.cpu().numpy(), b)
        o = r3.grouped_swiglu(s, got[4], got[1], wg[l], wu[l], wd[l], dev_status=st)
        torch.cuda.synchronize()
        assert st.item() == 0
        ragged = np.where(counts % 16 != 0)[0]
        experts = {int(np.argmax(counts)), int(np.argmin(counts)),
                   int(ragged[0]) if ragged.size else 0}
        for e in experts:
            lo, hi = int(offsets[e]), int(offsets[e + 1])
            tokens = torch.from_numpy(sor[lo:hi].astype(np.int64) // w.K).to(x.device)
            ref_o = O.swiglu_expert(f64(x[l][tokens]), LayerExperts(wg, l)[e],
                                    LayerExperts(wu, l)[e], LayerExperts(wd, l)[e])
            worst_o = max(worst_o, rel_err(f64(o[lo:hi]), ref_o))
        del o, got
    assert worst_o < tol, worst_o
    return worst_y, worst_ds, worst_o


def test_small_independent_blocks(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="blocks_bf16", T=300, d=256, E=16,
                     K=4, F=128)
    check_blocks(r3, w, 3, 300, 2e-2, rows_of_blocks=(0, 2))


def test_config5_48_blocks_full_size(r3):
    """Configuration 5: 48 MoE blocks (attention left out, so every block's input is a seeded
    synthetic tensor), T=16384, about 58 GB of expert weights resident.  Every block is held to
    the per-layer bar on 32 sampled tokens that the oracle evaluates from the equations, and on
    three blocks the dispatch is compared bit for bit and all rows of three experts (the largest,
    the smallest, one with a ragged last tile) row by row."""
    w = synth.WORKLOADS["c5_stack48"]
    free, _ = torch.cuda.mem_get_info()
    if free < 80e9:
        pytest.skip("needs about 75 GB of free device memory")
    worst_y, worst_ds, worst_o = check_blocks(r3, w, w.layers, 32, 2e-2, rows_of_blocks=(0, 23, 47))
    print(f"config 5: worst y err {worst_y:.2e}, worst dlogits err {worst_ds:.2e}, worst expert "
          f"row err {worst_o:.2e}")


def test_residual_chain_of_48_blocks_full_size(r3):
    """The same 48 blocks chained through residual connections.  The chain has no normalisation,
    so a perturbation of x_l is amplified block after block; only the stack output (with the
    tolerance derived in check_stack) and the router gradients of the first blocks, whose inputs
    have not drifted yet, are compared."""
    w = synth.WORKLOADS["c5_stack48"]
    free, _ = torch.cuda.mem_get_info()
    if free < 80e9:
        pytest.skip("needs about 75 GB of free device memory")
    sel = np.array([5, 4097, 9000, 16383])
    check_stack(r3, w, w.layers, sel, 2e-2, bf16_store, ds_layers=3)


def check_stack_train(r3, w, L, sel, tol, expert_grads=False):
    """r3_replay_stack_train against the oracle's exact chain on the tokens `sel` (all tokens when
    sel covers them: then dW_r is compared too)."""
    x0, dy, w_r, wg, wu, wd, idx = build_stack(w, L)
    s = r3.shape_of(w)
    st = r3.new_status("cuda")
    out = r3.replay_stack_train(s, L, x0, w_r, idx, wg, wu, wd, dy, dev_status=st,
                                expert_grads=expert_grads)
    x_out, dlogits, dx0, dw_r = out[:4]
    torch.cuda.synchronize()
    assert st.item() == 0
    idx_np = idx.cpu().to(torch.int64).numpy()
    layers = [(f64(w_r[l]), idx_np[l][sel], LayerExperts(wg, l), LayerExperts(wu, l),
               LayerExperts(wd, l)) for l in range(L)]
    ref = O.replay_stack_bwd_tokens(f64(x0)[sel], layers, f64(dy)[sel], store=bf16_store,
                                    expert_grads=expert_grads and len(sel) == w.T)
    # Only the stack output, a running sum stored L times, gets the random-walk term of
    # check_stack; every gradient (dlogits and dW_r of each block, dx0, expert weights) is held
    # to the flat per-layer bar.
    tol_x = tol + np.sqrt(L) * 2.0 ** -8
    err = lambda got, want: float(np.abs(got - want).max() / np.abs(want).max())
    measured = {"x_out": err(f64(x_out)[sel], ref["x_out"]), "dx0": err(f64(dx0)[sel], ref["dx0"]),
                "dlogits": max(err(f64(dlogits[l])[sel], ref["ds"][l]) for l in range(L))}
    if len(sel) == w.T:
        measured["dW_r"] = max(err(f64(dw_r[l]), ref["dw_r"][l]) for l in range(L))
        if expert_grads:
            measured["dW_experts"] = max(
                err(f64(out[4 + k][l]), np.stack([ref["dw_experts"][l][e][k] for e in range(w.E)]))
                for l in range(L) for k in range(3))
    print(f"{w.name} x{L} exact chain: " + ", ".join(f"{k} {v:.2e}" for k, v in measured.items()))
    assert measured.pop("x_out") < tol_x
    assert all(v < tol for v in measured.values()), measured
    # the forward half is r3_replay_stack's; a second run repeats the first bit for bit
    x_fwd, _ = r3.replay_stack(s, L, x0, w_r, idx, wg, wu, wd, dy)
    assert torch.equal(x_fwd, x_out)
    again = r3.replay_stack_train(s, L, x0, w_r, idx, wg, wu, wd, dy, expert_grads=expert_grads)
    assert all(torch.equal(a, b) for a, b in zip(out, again))
    return out


def test_small_stack_exact_backward_chain(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="stack_bwd", T=300, d=256, E=16,
                     K=4, F=128)
    check_stack_train(r3, w, 3, np.arange(300), 2e-2)


def test_small_stack_exact_backward_chain_with_expert_weight_gradients(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="stack_bwd_w", T=260, d=128, E=8,
                     K=2, F=136)
    check_stack_train(r3, w, 3, np.arange(260), 2e-2, expert_grads=True)


def test_one_block_stack_train_is_layer_train_plus_identity_path(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="stack_bwd1", T=200, d=256, E=16,
                     K=4, F=128)
    x0, dy, w_r, wg, wu, wd, idx = build_stack(w, 1)
    s = r3.shape_of(w)
    x1, dl, dx0, dwr, dwg, dwu, dwd = r3.replay_stack_train(s, 1, x0, w_r, idx, wg, wu, wd, dy,
                                                            expert_grads=True)
    y, ds, dx, dwr1, g1, u1, d1 = r3.replay_layer_train(s, x0, w_r[0], idx[0], wg[0], wu[0],
                                                        wd[0], dy, expert_grads=True)
    assert torch.equal(dl[0], ds) and torch.equal(dwr[0], dwr1)
    assert torch.equal(dwg[0], g1) and torch.equal(dwu[0], u1) and torch.equal(dwd[0], d1)
    scale = float(dx0.float().abs().max())
    assert (dx0.float() - (dy.float() + dx.float())).abs().max().item() <= scale * 2.0 ** -7


def test_four_blocks_of_config5_shape_exact_backward_chain(r3):
    """The configuration-5 block shape (T=16384, d=2048, E=128, K=8, F=768), four blocks chained,
    sampled tokens followed by the oracle through the whole forward and backward chain."""
    w = synth.WORKLOADS["c5_stack48"]
    free, _ = torch.cuda.mem_get_info()
    if free < 30e9:
        pytest.skip("needs about 25 GB of free device memory")
    check_stack_train(r3, w, 4, np.array([7, 4097, 9000, 16383]), 2e-2)
