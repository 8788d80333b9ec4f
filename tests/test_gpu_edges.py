"""Degenerate and boundary cases of the replayed layer on the GPU, each against the oracle:
no tokens, one token, K = 1 (gate 1, zero router gradient), K = E (every expert), all tokens on
one expert (127 empty experts, one expert spanning many token tiles), records wider than a byte
(int16, E > 256), token counts that straddle the 256-token chunks of the dispatch, and a
token count beyond what the one-launch dispatch can keep resident (three-launch path)."""
import numpy as np
import pytest
import torch

from oracle import r3_oracle as O
from paper_2510_11370_b200 import synth
from tests.helpers import Case, f32, f64, random_record, rel_err

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 1e-5


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import r3 as mod
    return mod


def layer_against_oracle(r3, case, tol, idx=None):
    if idx is not None:
        case.idx = idx
    s = r3.shape_of(case.w)
    c = case.cuda()
    st = r3.new_status("cuda")
    y, ds, g = r3.replay_layer(s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"], c["w_down"],
                               c["dy"], dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    ref = case.oracle_layer()
    assert rel_err(f64(g), ref["g"]) < 1e-5
    assert rel_err(f64(y), ref["y"]) < tol
    denom = np.abs(ref["ds"]).max()
    if denom > 0:
        assert rel_err(f64(ds), ref["ds"]) < tol
    else:
        assert float(ds.abs().max()) == 0.0
    return y, ds, g


def test_no_tokens_is_ok_and_launches_nothing(r3):
    s = r3.make_shape(0, 64, 8, 2, 64)
    e = lambda *sh, dt=torch.bfloat16: torch.empty(sh, dtype=dt, device="cuda")
    ws = r3.workspace(4096, "cuda")
    y, ds, g = r3.replay_layer(s, e(0, 64), e(8, 64, dt=torch.float32), e(0, 2, dt=torch.uint8),
                               e(8, 64, 64), e(8, 64, 64), e(8, 64, 64), e(0, 64), ws=ws)
    assert y.shape == (0, 64) and ds.shape == (0, 8)
    counts, offsets, ros, sor, _ = r3.permute(s, e(0, 2, dt=torch.uint8))
    torch.cuda.synchronize()
    assert counts.sum().item() == 0 and offsets.abs().sum().item() == 0


@pytest.mark.parametrize("act,tol", [("f32", TOL_F32), ("bf16", TOL_BF16)])
def test_one_token(r3, act, tol):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="one", T=1, d=128, E=16, K=4, F=64,
                     act=act)
    layer_against_oracle(r3, Case(w), tol)


def test_k1_gate_is_one_and_router_gradient_is_zero(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="k1", T=300, d=256, E=16, K=1, F=128)
    y, ds, g = layer_against_oracle(r3, Case(w), TOL_BF16)
    assert torch.all(g == 1.0) and torch.all(ds == 0.0)


def test_k_equals_e_uses_every_expert(r3):
    w = synth.scaled(synth.WORKLOADS["c1_tiny_fp32"], name="kE", T=130, d=64, E=8, K=8, F=64,
                     record="noise", sigma=0.5)
    case = Case(w)
    y, ds, g = layer_against_oracle(r3, case, TOL_F32)
    # K = M: the replay gate is the full softmax of the training logits
    full = torch.softmax(torch.from_numpy(case.s), dim=1).numpy()
    picked = np.take_along_axis(full, case.idx_np(), axis=1)
    assert rel_err(f64(g), picked) < 1e-5


def test_every_token_on_the_same_experts(r3):
    """K experts take all T tokens (T rows each, several 256-row token tiles), the others none."""
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="hot", T=700, d=256, E=32, K=2, F=128)
    case = Case(w)
    idx = torch.tensor([[5, 17]], dtype=torch.uint8).repeat(w.T, 1)
    y, ds, g = layer_against_oracle(r3, case, TOL_BF16, idx=idx)
    s = r3.shape_of(w)
    counts, offsets, _, _, _ = r3.permute(s, idx.cuda())
    c = counts.cpu().numpy()
    assert c[5] == w.T and c[17] == w.T and c.sum() == 2 * w.T


@pytest.mark.parametrize("act,tol", [("f32", TOL_F32), ("bf16", TOL_BF16)])
def test_int16_record_with_more_than_256_experts(r3, act, tol):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="wide", T=200, d=64, E=300, K=3, F=64,
                     act=act, sigma=0.2)
    assert w.idx_dtype == torch.int16
    layer_against_oracle(r3, Case(w), tol)


@pytest.mark.parametrize("T", [255, 256, 257, 513])
def test_dispatch_across_chunk_boundaries_is_bit_exact(r3, T):
    E, K = 24, 5
    idx = random_record(np.random.default_rng(T), T, E, K, torch.uint8)
    s = r3.make_shape(T, 8, E, K, 8)
    counts, offsets, ros, sor, _ = r3.permute(s, idx.cuda())
    rc, ro, rr, rs = O.permutation(idx.to(torch.int64).numpy(), E)
    assert np.array_equal(counts.cpu().numpy(), rc) and np.array_equal(offsets.cpu().numpy(), ro)
    assert np.array_equal(ros.cpu().numpy(), rr) and np.array_equal(sor.cpu().numpy(), rs)


def test_dispatch_of_more_chunks_than_fit_on_the_device_at_once(r3):
    """T / 256 chunk CTAs beyond the resident limit take the three-launch dispatch; the maps are
    checked against their defining properties (the oracle's stable sort at this size takes long)."""
    T, E, K = 400_000, 8, 2
    rng = np.random.default_rng(11)
    first = rng.integers(0, E, size=T)
    second = (first + rng.integers(1, E, size=T)) % E
    idx_np = np.stack([first, second], axis=1)
    idx = torch.from_numpy(idx_np.astype(np.uint8))
    s = r3.make_shape(T, 8, E, K, 8)
    counts, offsets, ros, sor, _ = r3.permute(s, idx.cuda())
    counts, offsets, ros, sor = (t.cpu().numpy() for t in (counts, offsets, ros, sor))
    assert np.array_equal(counts, np.bincount(idx_np.reshape(-1), minlength=E))
    assert np.array_equal(offsets, np.concatenate([[0], np.cumsum(counts)]))
    flat = ros.reshape(-1)
    assert np.array_equal(np.sort(flat), np.arange(T * K))              # a permutation
    assert np.array_equal(sor[flat], np.arange(T * K))                  # and its inverse
    expert_of_row = idx_np.reshape(-1)[sor]
    assert np.all(np.diff(expert_of_row) >= 0)                          # grouped by expert
    same = np.diff(expert_of_row) == 0
    assert np.all(np.diff(sor // K)[same] > 0)                          # stable within an expert


# ---- edge cases of the Update-stage backward entry points -------------------------------------
def train_against_oracle(r3, case, tol=TOL_BF16):
    w = case.w
    s = r3.shape_of(w)
    c = case.cuda()
    st = r3.new_status("cuda")
    y, ds, dx, dw_r, dwg, dwu, dwd = r3.replay_layer_train(
        s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"], c["w_down"], c["dy"],
        dev_status=st, expert_grads=True)
    torch.cuda.synchronize()
    assert st.item() == 0
    args = (f64(case.x), f64(case.w_r), case.idx_np(), f32(case.w_gate), f32(case.w_up),
            f32(case.w_down), f64(case.dy))
    ref = O.layer_bwd_input(*args)
    refw = O.layer_bwd_weights(*args)
    assert rel_err(f64(y), ref["y"]) < tol and rel_err(f64(dx), ref["dx"]) < tol
    if np.abs(ref["ds"]).max() > 0:
        assert rel_err(f64(ds), ref["ds"]) < tol and rel_err(f64(dw_r), ref["dw_r"]) < tol
    for k, got in enumerate((dwg, dwu, dwd)):
        full = np.stack([refw[e][k] for e in range(w.E)])
        assert rel_err(f64(got), full) < tol, k


def test_backward_with_a_record_wider_than_the_fused_finish(r3):
    """K = 12 > 8: the layer takes the four separate finishing kernels; the backward still gets
    its gates."""
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="bwd_k12", T=150, d=128, E=16, K=12,
                     F=64, sigma=0.3)
    train_against_oracle(r3, Case(w))


def test_backward_with_int16_record_and_many_experts(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="bwd_wide", T=400, d=64, E=300, K=3,
                     F=64, sigma=0.2)
    assert w.idx_dtype == torch.int16
    train_against_oracle(r3, Case(w))


def test_backward_of_one_token_and_of_one_hot_expert(r3):
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="bwd_one", T=1, d=128, E=16, K=4, F=64)
    train_against_oracle(r3, Case(w))
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="bwd_hot", T=333, d=256, E=32, K=2,
                     F=128)
    case = Case(w)
    case.idx = torch.tensor([[5, 17]], dtype=torch.uint8).repeat(w.T, 1)
    train_against_oracle(r3, case)


def test_backward_entry_points_reject_float32_and_accept_no_tokens(r3):
    e = lambda *sh, dt=torch.bfloat16: torch.empty(sh, dtype=dt, device="cuda")
    s0 = r3.make_shape(0, 64, 8, 2, 64)
    ws = r3.workspace(4096, "cuda")
    out = r3.replay_layer_train(s0, e(0, 64), e(8, 64, dt=torch.float32), e(0, 2, dt=torch.uint8),
                                e(8, 64, 64), e(8, 64, 64), e(8, 64, 64), e(0, 64), ws=ws)
    assert out[2].shape == (0, 64)
    w = synth.scaled(synth.WORKLOADS["c1_tiny_fp32"], name="bwd_f32", T=16, d=64, E=8, K=2, F=64)
    c = Case(w).cuda()
    s = r3.shape_of(w)
    with pytest.raises(r3.R3Error) as err:
        r3.replay_layer_train(s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"], c["w_down"],
                              c["dy"], ws=ws)
    assert err.value.code == r3.R3_ERR_UNSUPPORTED


def test_a_bounded_wait_that_runs_out_reports_timeout_and_leaves_the_context_usable(r3):
    """The pipelines of the tensor-core kernels never spin for ever: a barrier wait gives up
    after its clock limit, raises the abort flag and reports R3_DEV_TIMEOUT.  The self-test entry
    point makes exactly that happen (a barrier nothing signals, 200 000 clocks = about 0.1 ms)."""
    st = r3.new_status("cuda")
    out = r3.selftest_bounded_wait(200_000, dev_status=st)
    torch.cuda.synchronize()
    waited, second = int(out[2]), int(out[3])
    assert int(out[0]) == 0 and int(out[1]) == 1          # gave up, abort flag raised
    assert 200_000 <= waited < 50_000_000                 # after the limit, and not much later
    assert second == 0                                    # a later wait in the aborting CTA returns at once
    assert st.item() == r3.DEV_TIMEOUT
    # first error wins: a second run does not overwrite the word; a fresh word is set again
    r3.selftest_bounded_wait(1000, dev_status=st)
    assert st.item() == r3.DEV_TIMEOUT
    with pytest.raises(r3.R3Error):
        r3.selftest_bounded_wait(0)
    with pytest.raises(r3.R3Error):
        r3.selftest_bounded_wait(3_000_000_000)
    # the context is intact: an ordinary tensor-core call right after is clean and correct
    T, d, E, K = 300, 256, 32, 4
    x = torch.randn(T, d).to(torch.bfloat16).cuda()
    w = (torch.randn(E, d) * 0.1).to(torch.bfloat16).cuda()
    s = r3.make_shape(T, d, E, K, 8, router=torch.bfloat16)
    idx, logits = r3.capture_topk(s, x, w, want_logits=True)
    torch.cuda.synchronize()
    ref = x.float() @ w.float().T
    assert torch.allclose(logits, ref, atol=1e-2) and idx.shape == (T, K)


def test_gate_bwd_refuses_a_misaligned_dlogits_instead_of_faulting(r3):
    """dlogits rows are written in 16-byte pieces; a view that starts 4 bytes into an allocation
    is refused on the host (R3_ERR_INVALID_ARG), nothing is launched."""
    T, E, K = 64, 128, 8
    rng = np.random.default_rng(1)
    idx = random_record(rng, T, E, K, torch.uint8).cuda()
    g = torch.softmax(torch.randn(T, K), dim=1).cuda()
    dg = torch.randn(T, K).cuda()
    s = r3.make_shape(T, 8, E, K, 8)
    backing = torch.full((T * E + 4,), 7.0, dtype=torch.float32, device="cuda")
    view = backing[1:1 + T * E].view(T, E)
    assert view.data_ptr() % 16 == 4 and view.is_contiguous()
    with pytest.raises(r3.R3Error) as err:
        r3.replay_gate_bwd(s, g, dg, idx, dlogits=view)
    assert err.value.code == r3.R3_ERR_INVALID_ARG
    torch.cuda.synchronize()
    assert torch.all(backing == 7.0)
    ok = backing[4:4 + T * E].view(T, E)
    ds = r3.replay_gate_bwd(s, g, dg, idx, dlogits=ok)
    ref = O.replay_gate_bwd(g.cpu().numpy(), dg.cpu().numpy(), idx.cpu().to(torch.int64).numpy(), E)
    assert rel_err(ds.cpu().numpy(), ref) < TOL_F32


def test_inputs_written_by_the_kernel_just_before_the_call(r3):
    """The dispatch, the row copy and the layer's first kernels are launched so that they may begin
    before the kernel in front of them on the stream has ended, and the row copy fetches its token
    rows before its own dependency wait.  Here the activations (and the record) are produced by
    torch kernels enqueued directly in front of the call, without a synchronisation, forty times
    with other data, into the SAME buffers: a fetch that did not wait for its producer would pick
    up the rows of the round before."""
    T, d, E, K, F = 4096, 512, 32, 4, 64
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="chain", T=T, d=d, E=E, K=K, F=F)
    s = r3.shape_of(w)
    dev = torch.device("cuda", 0)
    g = torch.Generator(device=dev).manual_seed(3)
    base = torch.randn(T, d, generator=g, device=dev)
    x = torch.empty(T, d, dtype=torch.bfloat16, device=dev)
    idx = torch.empty(T, K, dtype=torch.uint8, device=dev)
    keys = torch.rand(40, T, E, generator=g, device=dev)
    ws = r3.workspace(r3.permute_workspace_bytes(s), dev)
    st = r3.new_status(dev)
    outs = []
    for r in range(40):
        # producers: one elementwise kernel for x, a top-k for the record, then the dispatch at once
        x.copy_((base * (r + 1)).to(torch.bfloat16))
        idx.copy_(keys[r].topk(K, dim=1).indices.to(torch.uint8))
        counts, offsets, ros, sor, xp = r3.permute(s, idx, x, ws=ws, dev_status=st)
        outs.append((idx.clone(), x.clone(), ros, xp))
    torch.cuda.synchronize()
    assert st.item() == 0
    for r, (idx_r, x_r, ros, xp) in enumerate(outs):
        _, _, ros_ref, sor_ref = O.permutation(idx_r.cpu().numpy().astype(np.int64), E)
        assert np.array_equal(ros.cpu().numpy(), ros_ref), r
        want = x_r[torch.from_numpy(sor_ref.astype(np.int64)).to(dev) // K]
        assert torch.equal(xp, want), r


def test_layer_fed_by_kernels_enqueued_directly_in_front_of_it(r3):
    """The same for the whole layer (its first kernels on both streams start under the tail of
    whatever precedes them): activations, upstream gradient and record rewritten by torch kernels
    in front of every call, twelve rounds into the same buffers and the same workspace; every
    round must give the bits of running its inputs alone after a synchronisation."""
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], name="chain_layer", T=3000, d=512, E=32,
                     K=4, F=128)
    case = Case(w, device="cuda")
    c = case.cuda()
    s = r3.shape_of(w)
    dev = torch.device("cuda", 0)
    st = r3.new_status(dev)
    ws = r3.workspace(r3.replay_layer_workspace_bytes(s), dev)
    g = torch.Generator(device=dev).manual_seed(9)
    keys = torch.rand(12, w.T, w.E, generator=g, device=dev)
    x, dy, idx = c["x"].clone(), c["dy"].clone(), c["idx"].clone()
    y = torch.empty_like(x)
    ds = torch.empty((w.T, w.E), dtype=torch.float32, device=dev)
    kept = []
    for r in range(12):
        x.copy_((c["x"].float() * (1.0 + 0.25 * r)).to(x.dtype))
        dy.copy_((c["dy"].float() * (1.0 - 0.05 * r)).to(dy.dtype))
        idx.copy_(keys[r].topk(w.K, dim=1).indices.to(idx.dtype))
        r3.replay_layer(s, x, c["w_r"], idx, c["w_gate"], c["w_up"], c["w_down"], dy, y=y,
                        dlogits=ds, ws=ws, dev_status=st)
        kept.append((x.clone(), dy.clone(), idx.clone(), y.clone(), ds.clone()))
    torch.cuda.synchronize()
    assert st.item() == 0
    for r, (xr, dyr, idxr, yr, dsr) in enumerate(kept):
        y1, ds1, _ = r3.replay_layer(s, xr, c["w_r"], idxr, c["w_gate"], c["w_up"], c["w_down"],
                                     dyr, dev_status=st)
        torch.cuda.synchronize()
        assert torch.equal(y1, yr) and torch.equal(ds1, dsr), r
