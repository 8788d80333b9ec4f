"""Update-stage backward to the layer input on the GPU against the oracle (Section 4.1, purpose
(b)): the expert input-gradient GEMMs with transposed weights, then the whole chain."""
import numpy as np
import pytest
import torch

from oracle import r3_oracle as O
from tests.helpers import f32, f64, rel_err

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import r3 as mod
    return mod


@pytest.mark.parametrize("T,d,E,K,F", [
    (256, 256, 4, 2, 128),        # a few full tiles
    (300, 2048, 16, 8, 768),      # the paper-like layer shape, ragged expert sizes
    (77, 136, 6, 3, 72),          # ragged d, F, experts smaller than a tile
    (1500, 512, 3, 2, 264),       # experts spanning many token tiles
])
def test_expert_input_gradient(r3, T, d, E, K, F):
    rng = np.random.default_rng(T + d)
    pop = rng.random(E) ** 2 + 0.01
    idx_np = np.argsort(-(rng.random((T, E)) * pop[None, :]), axis=1)[:, :K]
    _, offsets, ros, sor = O.permutation(idx_np, E)
    bf = torch.bfloat16
    x = torch.randn(T, d).to(bf)
    wg = (torch.randn(E, F, d) * 0.05).to(bf)
    wu = (torch.randn(E, F, d) * 0.05).to(bf)
    wd = (torch.randn(E, d, F) * 0.05).to(bf)
    xp = x[torch.from_numpy(sor.astype(np.int64)) // K].contiguous()
    dout = torch.randn(T * K, d).to(bf)
    # the forward's stored pre-activations (rounded to bf16 as the forward stores them)
    R = T * K
    a = torch.empty(R, F, dtype=bf)
    b = torch.empty(R, F, dtype=bf)
    ref = np.zeros((R, d))
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            continue
        xe = f64(xp[lo:hi])
        a[lo:hi] = torch.from_numpy(xe @ f64(wg[e]).T).to(bf)
        b[lo:hi] = torch.from_numpy(xe @ f64(wu[e]).T).to(bf)
        ref[lo:hi] = O.swiglu_expert_bwd_input(xe, f64(dout[lo:hi]), f32(wg[e]), f32(wu[e]), f32(wd[e]))
    s = r3.make_shape(T, d, E, K, F)
    st = r3.new_status("cuda")
    dxp = r3.grouped_swiglu_bwd_input(s, dout.cuda(), a.cuda(), b.cuda(),
                                      torch.from_numpy(offsets).cuda(), wg.cuda(), wu.cuda(),
                                      wd.cuda(), dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    err = rel_err(f64(dxp), ref)
    assert err < TOL_BF16, err
    dxp2 = r3.grouped_swiglu_bwd_input(s, dout.cuda(), a.cuda(), b.cuda(),
                                       torch.from_numpy(offsets).cuda(), wg.cuda(), wu.cuda(),
                                       wd.cuda())
    assert torch.equal(dxp, dxp2)


def test_training_forward_keeps_the_pre_activations(r3):
    """r3_grouped_swiglu_train: same o as the plain forward, plus a = xp Wg^T and b = xp Wu^T."""
    T, d, E, K, F = 600, 512, 8, 2, 264
    rng = np.random.default_rng(3)
    idx_np = np.argsort(rng.random((T, E)), axis=1)[:, :K]
    _, offsets, ros, sor = O.permutation(idx_np, E)
    bf = torch.bfloat16
    x = torch.randn(T, d, generator=torch.Generator().manual_seed(1)).to(bf)
    wg = (torch.randn(E, F, d) * 0.05).to(bf).cuda()
    wu = (torch.randn(E, F, d) * 0.05).to(bf).cuda()
    wd = (torch.randn(E, d, F) * 0.05).to(bf).cuda()
    xp = x[torch.from_numpy(sor.astype(np.int64)) // K].contiguous().cuda()
    off = torch.from_numpy(offsets).cuda()
    s = r3.make_shape(T, d, E, K, F)
    st = r3.new_status("cuda")
    o, a, b = r3.grouped_swiglu_train(s, xp, off, wg, wu, wd, dev_status=st)
    o_plain = r3.grouped_swiglu(s, xp, off, wg, wu, wd)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert torch.equal(o, o_plain)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        xe = f64(xp[lo:hi])
        ref_a, ref_b = xe @ f64(wg[e]).T, xe @ f64(wu[e]).T
        assert rel_err(f64(a[lo:hi]), ref_a) < 1e-2     # bf16 storage: 2^-9 relative
        assert rel_err(f64(b[lo:hi]), ref_b) < 1e-2


def test_scale_rows_and_input_grad_finish_against_definitions(r3):
    """The two memory-bound steps alone, on random inputs, against their defining sums."""
    T, d, E, K = 333, 136, 12, 3
    rng = np.random.default_rng(9)
    idx_np = np.argsort(rng.random((T, E)), axis=1)[:, :K]
    _, offsets, ros, sor = O.permutation(idx_np, E)
    bf = torch.bfloat16
    dy = torch.randn(T, d).to(bf)
    x = torch.randn(T, d).to(bf)
    gates = torch.rand(T, K)
    w_r = torch.randn(E, d) * 0.1
    dxp = torch.randn(T * K, d).to(bf)
    ds = torch.zeros(T, E)
    ds.scatter_(1, torch.from_numpy(idx_np), torch.randn(T, K))
    s = r3.make_shape(T, d, E, K, 64)
    ros_t, sor_t = torch.from_numpy(ros).cuda(), torch.from_numpy(sor).cuda()
    dout = r3.scale_rows(s, dy.cuda(), gates.cuda(), ros_t)
    ref = np.zeros((T * K, d))
    for t in range(T):
        for j in range(K):
            ref[ros[t, j]] = float(gates[t, j]) * f64(dy[t])
    assert rel_err(f64(dout), ref) < 4e-3                  # one bf16 rounding
    dx, dw_r = r3.input_grad_finish(s, dxp.cuda(), ros_t, sor_t, torch.from_numpy(offsets).cuda(),
                                    ds.cuda(), torch.from_numpy(idx_np.astype(np.uint8)).cuda(),
                                    x.cuda(), w_r.cuda())
    ref_dx = f64(dxp)[ros].sum(axis=1) + f64(ds) @ f64(w_r)
    assert rel_err(f64(dx), ref_dx) < 4e-3
    assert rel_err(f64(dw_r), f64(ds).T @ f64(x)) < 1e-5


@pytest.mark.parametrize("name,T,d,E,K,F", [
    ("bwd_a", 300, 256, 16, 4, 128),
    ("bwd_b", 1000, 512, 8, 2, 264),
    ("bwd_k1", 200, 256, 16, 1, 128),
])
def test_layer_backward_to_input_and_router_weight(r3, name, T, d, E, K, F):
    from paper_2510_11370_b200 import synth
    from tests.helpers import Case
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name=name, T=T, d=d, E=E, K=K, F=F)
    case = Case(w)
    c = case.cuda()
    s = r3.shape_of(w)
    st = r3.new_status("cuda")
    y, ds, dx, dw_r = r3.replay_layer_train(s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"],
                                            c["w_down"], c["dy"], dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    ref = O.layer_bwd_input(f64(case.x), f64(case.w_r), case.idx_np(), f32(case.w_gate),
                            f32(case.w_up), f32(case.w_down), f64(case.dy))
    assert rel_err(f64(y), ref["y"]) < TOL_BF16
    assert rel_err(f64(dx), ref["dx"]) < TOL_BF16
    if K > 1:
        assert rel_err(f64(ds), ref["ds"]) < TOL_BF16
        assert rel_err(f64(dw_r), ref["dw_r"]) < TOL_BF16
    else:
        assert float(ds.abs().max()) == 0.0 and float(dw_r.abs().max()) == 0.0
    # the forward half is r3_replay_layer's, bit for bit, and a second run repeats the first
    y0, ds0, _ = r3.replay_layer(s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"],
                                 c["w_down"], c["dy"])
    assert torch.equal(y, y0) and torch.equal(ds, ds0)
    y2, ds2, dx2, dw2 = r3.replay_layer_train(s, c["x"], c["w_r"], c["idx"], c["w_gate"],
                                              c["w_up"], c["w_down"], c["dy"])
    assert torch.equal(dx, dx2) and torch.equal(dw_r, dw2)


def test_layer_backward_full_size_sampled_tokens(r3):
    """The benchmark layer (T=4096, d=2048, E=128, K=8, F=768): dx of sampled tokens and dW_r rows
    of sampled experts against the oracle evaluated on those tokens / experts only."""
    from paper_2510_11370_b200 import synth
    from tests.helpers import Case
    w = synth.WORKLOADS["c2_layer_bf16"]
    case = Case(w)
    c = case.cuda()
    s = r3.shape_of(w)
    st = r3.new_status("cuda")
    y, ds, dx, dw_r = r3.replay_layer_train(s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"],
                                            c["w_down"], c["dy"], dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    sel = np.array([0, 1, 255, 256, 1777, 2048, 3000, 4095])
    idx_sel = case.idx_np()[sel]

    class Experts:
        def __init__(self, t): self.t = t
        def __len__(self): return self.t.shape[0]
        def __getitem__(self, i): return f32(self.t[int(i)])

    ref = O.layer_bwd_input(f64(case.x)[sel], f64(case.w_r), idx_sel, Experts(case.w_gate),
                            Experts(case.w_up), Experts(case.w_down), f64(case.dy)[sel])
    scale = np.abs(ref["dx"]).max()
    assert np.abs(f64(dx)[sel] - ref["dx"]).max() / scale < TOL_BF16
    assert np.abs(f64(ds)[sel] - ref["ds"]).max() / np.abs(ref["ds"]).max() < TOL_BF16
    # dW_r = ds^T x uses every token: check it from the device's own ds (already compared above
    # on samples, and against the oracle in full at the small sizes)
    ref_dw = f64(ds).T @ f64(case.x)
    assert rel_err(f64(dw_r), ref_dw) < 1e-5


@pytest.mark.parametrize("T,d,E,K,F", [
    (256, 256, 4, 2, 256),        # full tiles, every expert a multiple of 16 rows or not
    (300, 2048, 16, 8, 768),      # the paper-like layer shape, ragged expert sizes
    (77, 136, 6, 3, 72),          # ragged d, F; experts smaller than one 64-row block
    (1500, 512, 3, 2, 264),       # experts spanning many 64-row blocks
    (2300, 328, 3, 2, 520),       # over 1024 rows per expert: the 256-row tile, ragged d and F
    (2100, 512, 2, 1, 256),       # the 256-row tile with full tiles only
])
def test_expert_weight_gradients(r3, T, d, E, K, F):
    """r3_grouped_swiglu_bwd: dW_gate, dW_up, dW_down of every expert against the oracle, fed the
    same stored bf16 pre-activations; an expert without rows gets zeros."""
    rng = np.random.default_rng(T + d + 1)
    pop = rng.random(E) ** 2 + 0.01
    pop[E - 1] = 0.0                                  # the last expert is never picked
    idx_np = np.argsort(-(rng.random((T, E)) * pop[None, :] + (pop[None, :] > 0)), axis=1)[:, :K]
    assert not np.any(idx_np == E - 1)
    _, offsets, ros, sor = O.permutation(idx_np, E)
    bf = torch.bfloat16
    g = torch.Generator().manual_seed(T)
    x = torch.randn(T, d, generator=g).to(bf)
    wg = (torch.randn(E, F, d, generator=g) * 0.05).to(bf)
    wu = (torch.randn(E, F, d, generator=g) * 0.05).to(bf)
    wd = (torch.randn(E, d, F, generator=g) * 0.05).to(bf)
    xp = x[torch.from_numpy(sor.astype(np.int64)) // K].contiguous()
    dout = torch.randn(T * K, d, generator=g).to(bf)
    R = T * K
    a = torch.empty(R, F, dtype=bf)
    b = torch.empty(R, F, dtype=bf)
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        xe = f64(xp[lo:hi])
        a[lo:hi] = torch.from_numpy(xe @ f64(wg[e]).T).to(bf)
        b[lo:hi] = torch.from_numpy(xe @ f64(wu[e]).T).to(bf)
    s = r3.make_shape(T, d, E, K, F)
    st = r3.new_status("cuda")
    args = (s, xp.cuda(), dout.cuda(), a.cuda(), b.cuda(), torch.from_numpy(offsets).cuda(),
            wg.cuda(), wu.cuda(), wd.cuda())
    dxp, dwg, dwu, dwd = r3.grouped_swiglu_bwd(*args, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    dxp_only = r3.grouped_swiglu_bwd_input(s, *args[2:])
    assert torch.equal(dxp, dxp_only)
    got = [f64(dwg), f64(dwu), f64(dwd)]
    scale = [0.0, 0.0, 0.0]
    refs = []
    for e in range(E):
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        ref = O.swiglu_expert_bwd_weights(f64(xp[lo:hi]), f64(dout[lo:hi]), f32(wg[e]), f32(wu[e]),
                                          f32(wd[e]))
        refs.append(ref)
        scale = [max(sc, float(np.abs(r).max())) for sc, r in zip(scale, ref)]
    for e in range(E):
        for k in range(3):
            err = np.abs(got[k][e] - refs[e][k]).max() / scale[k]
            assert err < TOL_BF16, (e, k, err)
    assert float(dwg[E - 1].abs().max()) == 0.0 and float(dwd[E - 1].abs().max()) == 0.0
    again = r3.grouped_swiglu_bwd(*args)
    assert all(torch.equal(p, q) for p, q in zip((dxp, dwg, dwu, dwd), again))


@pytest.mark.parametrize("T,d,E,K,F", [
    (700, 256, 16, 4, 136),       # 175 rows per expert: the 128-row weight-gradient tile
    (2200, 320, 4, 2, 264),       # 1100 rows per expert: the 256-row tile, ragged d and F
])
def test_layer_backward_with_expert_weight_gradients(r3, T, d, E, K, F):
    from paper_2510_11370_b200 import synth
    from tests.helpers import Case
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="bwd_w", T=T, d=d, E=E, K=K, F=F)
    case = Case(w)
    c = case.cuda()
    s = r3.shape_of(w)
    st = r3.new_status("cuda")
    y, ds, dx, dw_r, dwg, dwu, dwd = r3.replay_layer_train(
        s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"], c["w_down"], c["dy"],
        dev_status=st, expert_grads=True)
    torch.cuda.synchronize()
    assert st.item() == 0
    ref = O.layer_bwd_weights(f64(case.x), f64(case.w_r), case.idx_np(), f32(case.w_gate),
                              f32(case.w_up), f32(case.w_down), f64(case.dy))
    for k, got in enumerate((dwg, dwu, dwd)):
        full = np.stack([ref[e][k] for e in range(w.E)])
        assert rel_err(f64(got), full) < TOL_BF16
    y0, ds0, dx0, dwr0 = r3.replay_layer_train(s, c["x"], c["w_r"], c["idx"], c["w_gate"],
                                               c["w_up"], c["w_down"], c["dy"])
    assert torch.equal(dx, dx0) and torch.equal(dw_r, dwr0) and torch.equal(y, y0)


def test_expert_weight_gradients_paper_shape_sampled_experts(r3):
    """The 256-row weight-gradient tile at the paper-like layer shape (16384 tokens, 1024 rows per
    expert on average, d=2048, F=768): the experts with the most and the fewest rows and one in
    between, each of its three gradients in full against the oracle.  The inputs are drawn on the
    device by torch; the stored pre-activations of the checked experts are formed on the host in
    float64 and rounded to bf16 (those of the other experts are random: their gradients are not
    looked at)."""
    T, d, E, K, F = 16384, 2048, 128, 8, 768
    R = T * K
    dev = torch.device("cuda", 0)
    bf = torch.bfloat16
    rng = np.random.default_rng(11)
    idx_np = np.argsort(rng.random((T, E)) * (0.5 + rng.random(E))[None, :], axis=1)[:, :K]
    counts, offsets, ros, sor = O.permutation(idx_np, E)
    g = torch.Generator(device=dev).manual_seed(11)
    x = torch.randn(T, d, generator=g, device=dev).to(bf)
    wg = (torch.randn(E, F, d, generator=g, device=dev) * 0.05).to(bf)
    wu = (torch.randn(E, F, d, generator=g, device=dev) * 0.05).to(bf)
    wd = (torch.randn(E, d, F, generator=g, device=dev) * 0.05).to(bf)
    dout = torch.randn(R, d, generator=g, device=dev).to(bf)
    a = torch.randn(R, F, generator=g, device=dev).to(bf)
    b = torch.randn(R, F, generator=g, device=dev).to(bf)
    xp = x[torch.from_numpy(sor.astype(np.int64)).to(dev) // K].contiguous()
    order = np.argsort(counts)
    picks = [int(order[-1]), int(order[0]), int(order[E // 2])]
    assert counts[picks[0]] > 1024          # the 256-row tile is the one that runs
    host = {}
    for e in picks:
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        xe = f64(xp[lo:hi].cpu())
        a[lo:hi] = torch.from_numpy(xe @ f64(wg[e].cpu()).T).to(bf).to(dev)
        b[lo:hi] = torch.from_numpy(xe @ f64(wu[e].cpu()).T).to(bf).to(dev)
        host[e] = (xe, f64(dout[lo:hi].cpu()))
    s = r3.make_shape(T, d, E, K, F)
    st = r3.new_status(dev)
    dxp, dwg, dwu, dwd = r3.grouped_swiglu_bwd(s, xp, dout, a, b, torch.from_numpy(offsets).to(dev),
                                               wg, wu, wd, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    worst = 0.0
    for e in picks:
        xe, de = host[e]
        ref = O.swiglu_expert_bwd_weights(xe, de, f32(wg[e].cpu()), f32(wu[e].cpu()),
                                          f32(wd[e].cpu()))
        for k, got in enumerate((dwg, dwu, dwd)):
            err = rel_err(f64(got[e].cpu()), ref[k])
            worst = max(worst, err)
            assert err < TOL_BF16, (e, k, err, int(counts[e]))
    print(f"weight gradients at T={T}: rows of the checked experts "
          f"{[int(counts[e]) for e in picks]}, worst error {worst:.2e}")
