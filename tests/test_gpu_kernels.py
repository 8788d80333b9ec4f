"""Per-kernel parity of the CUDA library (through the C ABI) against the CPU oracle.

Integer outputs (records on exact data, counts, offsets, permutation maps, permuted rows) must be
bit-exact; floating-point outputs are judged by max|err| / max|ref| (2e-2 for bf16 storage,
1e-5 for float32)."""
import numpy as np
import pytest
import torch

from oracle import r3_oracle as O
from tests.helpers import f32, f64, random_record, rel_err

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 1e-5


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import r3 as mod
    return mod


def idx_dtype(E):
    return torch.uint8 if E <= 256 else torch.int16


# ------------------------------------------------------------------ replay gate fwd / bwd
@pytest.mark.parametrize("T,E,K", [(1, 8, 2), (513, 8, 1), (1000, 128, 8), (777, 130, 5),
                                   (300, 300, 32), (65, 64, 40), (4096, 128, 8), (31, 1024, 3)])
def test_replay_gate_fwd_bwd(r3, T, E, K):
    rng = np.random.default_rng(T * 31 + E)
    logits = torch.from_numpy(rng.standard_normal((T, E)).astype(np.float32) * 3)
    idx = random_record(rng, T, E, K, idx_dtype(E))
    dg = torch.from_numpy(rng.standard_normal((T, K)).astype(np.float32))
    s = r3.make_shape(T, 8, E, K, 8, idx=idx_dtype(E))
    st = r3.new_status("cuda")
    g = r3.replay_gate_fwd(s, logits.cuda(), idx.cuda(), dev_status=st)
    ds = r3.replay_gate_bwd(s, g, dg.cuda(), idx.cuda())
    torch.cuda.synchronize()
    assert st.item() == 0
    g_ref = O.replay_gate(logits.numpy(), idx.numpy())
    assert rel_err(g.cpu().numpy(), g_ref) < TOL_F32
    assert np.allclose(g.cpu().numpy().sum(axis=1), 1.0, atol=1e-5)
    ds_ref = O.replay_gate_bwd(g_ref, dg.numpy(), idx.to(torch.int64).numpy(), E)
    got = ds.cpu().numpy()
    assert rel_err(got, ds_ref) < TOL_F32
    off = np.ones((T, E), dtype=bool)
    off[np.arange(T)[:, None], idx.to(torch.int64).numpy()] = False
    assert np.all(got[off] == 0)                      # exact zeros off the mask


def test_replay_gate_flags_bad_records(r3):
    T, E, K = 64, 16, 4
    rng = np.random.default_rng(0)
    logits = torch.randn(T, E).cuda()
    idx = random_record(rng, T, E, K, torch.uint8)
    idx[5, 2] = idx[5, 0]                             # duplicate
    s = r3.make_shape(T, 8, E, K, 8)
    st = r3.new_status("cuda")
    g = r3.replay_gate_fwd(s, logits, idx.cuda(), dev_status=st)
    assert st.item() == r3.DEV_DUP_INDEX
    assert torch.all(g[5] == 0) and torch.allclose(g[6].sum(), torch.tensor(1.0, device="cuda"))
    idx = random_record(rng, T, E, K, torch.uint8)
    idx[9, 1] = 200                                   # out of range
    st = r3.new_status("cuda")
    g = r3.replay_gate_fwd(s, logits, idx.cuda(), dev_status=st)
    assert st.item() == r3.DEV_BAD_INDEX and torch.all(g[9] == 0)


# ------------------------------------------------------------------ permute
@pytest.mark.parametrize("T,E,K,d", [(1, 4, 2, 8), (255, 8, 2, 128), (256, 8, 8, 64),
                                     (257, 128, 8, 256), (1000, 1000, 3, 8), (5000, 128, 8, 2048),
                                     (70000, 64, 4, 32)])
@pytest.mark.parametrize("act", [torch.bfloat16, torch.float32])
def test_permute_bit_exact(r3, T, E, K, d, act):
    rng = np.random.default_rng(T + E)
    # skewed popularity so that some experts are empty and some are very large
    pop = rng.random(E) ** 4
    keys = rng.random((T, E)) * pop[None, :]
    idx_np = np.argsort(-keys, axis=1)[:, :K]
    idx = torch.from_numpy(idx_np).to(idx_dtype(E))
    x = torch.randn(T, d).to(act)
    s = r3.make_shape(T, d, E, K, 8, act=act, idx=idx_dtype(E))
    st = r3.new_status("cuda")
    out1 = r3.permute(s, idx.cuda(), x.cuda(), dev_status=st)
    out2 = r3.permute(s, idx.cuda(), x.cuda(), dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    counts, offsets, ros, sor = O.permutation(idx_np, E)
    for got, ref in zip(out1[:4], (counts, offsets, ros, sor)):
        assert np.array_equal(got.cpu().numpy(), ref)
    xp_ref = x[torch.from_numpy(sor.astype(np.int64)) // K]
    assert torch.equal(out1[4].cpu(), xp_ref)
    for a, b in zip(out1, out2):                      # run-to-run bitwise equality
        assert torch.equal(a, b)


def test_permute_drops_and_flags_invalid_pairs(r3):
    T, E, K = 300, 16, 4
    rng = np.random.default_rng(3)
    idx = random_record(rng, T, E, K, torch.uint8)
    idx[7, 3] = 99
    s = r3.make_shape(T, 8, E, K, 8)
    st = r3.new_status("cuda")
    counts, offsets, ros, sor, _ = r3.permute(s, idx.cuda(), dev_status=st)
    assert st.item() == r3.DEV_BAD_INDEX
    assert ros[7, 3].item() == -1 and counts.sum().item() == T * K - 1
    assert offsets[-1].item() == T * K - 1


# ------------------------------------------------------------------ combine / dgates
@pytest.mark.parametrize("T,K,d,act,tol", [(37, 2, 128, torch.float32, TOL_F32),
                                           (300, 8, 2048, torch.bfloat16, TOL_BF16),
                                           (129, 3, 72, torch.bfloat16, TOL_BF16),
                                           (64, 12, 520, torch.float32, TOL_F32)])
def test_combine_and_dgates(r3, T, K, d, act, tol):
    rng = np.random.default_rng(T)
    E = 16
    idx_np = random_record(rng, T, E, K, torch.int64).numpy()
    _, _, ros, sor = O.permutation(idx_np, E)
    o = torch.randn(T * K, d).to(act)
    dy = torch.randn(T, d).to(act)
    gates = torch.softmax(torch.randn(T, K), dim=1)
    s = r3.make_shape(T, d, E, K, 8, act=act)
    ros_c = torch.from_numpy(ros).cuda()
    y = r3.combine(s, o.cuda(), ros_c, gates.cuda())
    dg = r3.combine_bwd_gates(s, dy.cuda(), o.cuda(), ros_c)
    eo = f64(o)[ros.astype(np.int64)]                  # [T, K, d] expert output of each slot
    y_ref = np.einsum("tk,tkd->td", f64(gates), eo)
    assert rel_err(f64(y), y_ref) < tol
    assert rel_err(f64(dg), O.dgates(f64(dy), eo)) < TOL_F32 * 10
    y2 = r3.combine(s, o.cuda(), ros_c, gates.cuda())
    assert torch.equal(y, y2)


# ------------------------------------------------------------------ fused finish
@pytest.mark.parametrize("T,E,K,d,act,tol,residual", [
    (37, 8, 2, 128, torch.float32, TOL_F32, False),
    (300, 128, 8, 2048, torch.bfloat16, TOL_BF16, False),
    (129, 16, 3, 72, torch.bfloat16, TOL_BF16, True),
    (513, 10, 8, 520, torch.float32, TOL_F32, True),
    (1, 4, 1, 8, torch.bfloat16, TOL_BF16, False),
])
def test_replay_finish_matches_the_four_kernels_and_the_oracle(r3, T, E, K, d, act, tol, residual):
    """Gate + combine + both gradients in one pass: gates and y bit-identical to the separate
    calls, dlogits equal to theirs up to the summation order of the gate gradient, and everything
    within tolerance of the oracle's Eq. replay_gate / replay_output / gradient."""
    rng = np.random.default_rng(T + K)
    idx_t = random_record(rng, T, E, K, torch.uint8)
    idx_np = idx_t.to(torch.int64).numpy()
    _, _, ros, _ = O.permutation(idx_np, E)
    logits = (torch.randn(T, E) * 2).float()
    o = torch.randn(T * K, d).to(act)
    dy = torch.randn(T, d).to(act)
    res = torch.randn(T, d).to(act) if residual else None
    s = r3.make_shape(T, d, E, K, 8, act=act)
    ros_c = torch.from_numpy(ros).cuda()
    st = r3.new_status("cuda")
    y, g, ds = r3.replay_finish(s, logits.cuda(), idx_t.cuda(), o.cuda(), ros_c, dy.cuda(),
                                residual=None if res is None else res.cuda(), dev_status=st)
    assert st.item() == 0
    # the four kernels
    g4 = r3.replay_gate_fwd(s, logits.cuda(), idx_t.cuda())
    y4 = (r3.combine_residual(s, o.cuda(), ros_c, g4, res.cuda()) if residual
          else r3.combine(s, o.cuda(), ros_c, g4))
    dg4 = r3.combine_bwd_gates(s, dy.cuda(), o.cuda(), ros_c)
    ds4 = r3.replay_gate_bwd(s, g4, dg4, idx_t.cuda())
    assert torch.equal(g, g4) and torch.equal(y, y4)
    assert rel_err(f64(ds), f64(ds4)) < TOL_F32
    y_b, g_b, ds_b = r3.replay_finish(s, logits.cuda(), idx_t.cuda(), o.cuda(), ros_c, dy.cuda(),
                                      residual=None if res is None else res.cuda())
    assert torch.equal(y, y_b) and torch.equal(g, g_b) and torch.equal(ds, ds_b)   # reproducible
    # the oracle
    g_ref = O.replay_gate(f64(logits), idx_np)
    eo = f64(o)[ros.astype(np.int64)]
    y_ref = np.einsum("tk,tkd->td", g_ref, eo) + (f64(res) if residual else 0.0)
    ds_ref = O.replay_gate_bwd(g_ref, O.dgates(f64(dy), eo), idx_np, E)
    assert rel_err(f64(g), g_ref) < TOL_F32
    assert rel_err(f64(y), y_ref) < tol
    assert rel_err(f64(ds), ds_ref) < max(tol, TOL_F32 * 10)


def test_replay_finish_flags_bad_records_and_rejects_wide_k(r3):
    T, E, K, d = 64, 16, 4, 64
    rng = np.random.default_rng(5)
    idx = random_record(rng, T, E, K, torch.uint8)
    idx[3, 1] = idx[3, 0]                               # duplicate
    _, _, ros, _ = O.permutation(random_record(rng, T, E, K, torch.int64).numpy(), E)
    s = r3.make_shape(T, d, E, K, 8)
    st = r3.new_status("cuda")
    y, g, ds = r3.replay_finish(s, torch.randn(T, E).cuda(), idx.cuda(),
                                torch.randn(T * K, d).bfloat16().cuda(),
                                torch.from_numpy(ros).cuda(), torch.randn(T, d).bfloat16().cuda(),
                                dev_status=st)
    assert st.item() == r3.DEV_DUP_INDEX
    assert torch.all(g[3] == 0) and torch.all(ds[3] == 0) and torch.all(y[3] == 0)
    wide = r3.make_shape(T, d, E, 12, 8)
    with pytest.raises(r3.R3Error) as ei:
        r3.replay_finish(wide, torch.randn(T, E).cuda(), torch.zeros(T, 12, dtype=torch.uint8).cuda(),
                         torch.randn(T * 12, d).bfloat16().cuda(),
                         torch.zeros(T, 12, dtype=torch.int32).cuda(),
                         torch.randn(T, d).bfloat16().cuda())
    assert ei.value.code == 2


# ------------------------------------------------------------------ capture: logits + TopKMask
def plant_signed_zeros(x, w):
    """Logits that are zero with either sign.  Token 7 is all +0 and token 9 all -0, expert 3 has
    only negative and expert 1 only positive weights, so the products of those tokens are zeros of
    both signs and a sum of them may come out as -0.0 or +0.0 depending on the order and the unit
    that adds them.  TopKMask orders VALUES: -0.0 and +0.0 are the same logit, a tie, and the
    lower expert index wins (for tokens 7 and 9 the record is 0, 1, ..., K-1)."""
    x[7] = 0.0
    x[9] = -0.0
    w[3] = -1.0
    w[1] = 1.0
    w[11] = -2.0


@pytest.mark.parametrize("act,rw", [(torch.float32, torch.float32), (torch.bfloat16, torch.float32),
                                    (torch.bfloat16, torch.bfloat16)])
def test_capture_exact_arithmetic_with_planted_ties(r3, act, rw):
    """Small-integer data: every partial sum is exact in float32, so the record must equal the
    oracle's bit for bit, including the slot order and the tie rule."""
    T, d, E, K = 333, 64, 24, 6
    rng = np.random.default_rng(5)
    x = torch.from_numpy(rng.integers(-3, 4, (T, d)).astype(np.float32)).to(act)
    w = torch.from_numpy(rng.integers(-2, 3, (E, d)).astype(np.float32)).to(rw)
    w[5] = w[2]
    w[17] = w[2]                                       # three experts always tie
    plant_signed_zeros(x, w)
    s = r3.make_shape(T, d, E, K, 8, act=act, router=rw)
    idx, logits = r3.capture_topk(s, x.cuda(), w.cuda(), want_logits=True)
    ref_s = O.router_logits(f64(x), f64(w))
    assert np.array_equal(logits.cpu().numpy().astype(np.float64), ref_s)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), O.topk_indices(ref_s, K))


@pytest.mark.parametrize("rw", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("T,d,E,K", [(333, 64, 32, 6), (1000, 200, 128, 8), (130, 2048, 256, 16)])
def test_capture_tensor_core_exact_arithmetic_with_planted_ties(r3, rw, T, d, E, K):
    """The tcgen05 router kernel (bf16 activations, E a multiple of 16) on small-integer data:
    sums are exact, so logits and record must equal the oracle's bit for bit, ties included.
    float32 weights go through the three-plane split (the integers sit entirely in the top plane)."""
    rng = np.random.default_rng(T + E)
    x = torch.from_numpy(rng.integers(-3, 4, (T, d)).astype(np.float32)).to(torch.bfloat16)
    w = torch.from_numpy(rng.integers(-2, 3, (E, d)).astype(np.float32)).to(rw)
    w[5] = w[2]
    w[17] = w[2]
    w[E - 1] = w[0]
    plant_signed_zeros(x, w)
    s = r3.make_shape(T, d, E, K, 8, router=rw)
    idx, logits = r3.capture_topk_ws(s, 1, x.cuda(), w.cuda(), want_logits=True)
    ref_s = O.router_logits(f64(x), f64(w))
    assert np.array_equal(logits.cpu().numpy().astype(np.float64), ref_s)
    assert np.array_equal(idx.cpu().numpy().astype(np.int64), O.topk_indices(ref_s, K))


@pytest.mark.parametrize("T,d,E,K,L", [(4096, 2048, 128, 8, 1), (300, 520, 64, 4, 3),
                                       (129, 2048, 256, 8, 2)])
def test_capture_tensor_core_fp32_router_weights_keep_fp32_accuracy(r3, T, d, E, K, L):
    x = torch.randn(L, T, d).to(torch.bfloat16)
    w = torch.randn(L, E, d) * 0.02
    s = r3.make_shape(T, d, E, K, 8)
    assert r3.capture_topk_workspace_bytes(s, L) >= L * 3 * E * d * 2
    idx, logits = r3.capture_topk_ws(s, L, x.cuda(), w.cuda(), want_logits=True)
    near = 0
    for l in range(L):
        ref_s = O.router_logits(f64(x[l]), f64(w[l]))
        assert rel_err(logits[l].cpu().numpy(), ref_s) < TOL_F32
        near += check_record_against_logits(idx[l].cpu().numpy(), ref_s, K)
    assert near < 0.05 * L * T
    # logits only / record only give the same values
    only_idx, _ = r3.capture_topk_ws(s, L, x.cuda(), w.cuda())
    assert torch.equal(only_idx, idx)


def check_record_against_logits(idx_gpu, s_ref, K, tau=1e-3):
    """Margin rule for floating-point near-ties: where the oracle's K-th and (K+1)-th logits are
    at least tau apart the sets must be equal; elsewhere the chosen set must be within tau of
    optimal.  Returns the number of near-tie tokens."""
    T, E = s_ref.shape
    srt = -np.sort(-s_ref, axis=1)
    margin = srt[:, K - 1] - srt[:, K] if K < E else np.full(T, np.inf)
    ref = O.topk_indices(s_ref, K)
    got = np.asarray(idx_gpu, dtype=np.int64)
    safe = margin >= tau
    assert np.array_equal(np.sort(got[safe], axis=1), np.sort(ref[safe], axis=1))
    for t in np.nonzero(~safe)[0]:
        chosen = set(got[t].tolist())
        assert len(chosen) == K
        lo = min(s_ref[t, i] for i in chosen)
        hi = max(s_ref[t, i] for i in range(E) if i not in chosen)
        assert lo >= hi - tau
    # slot order: descending logits (up to tau)
    sel = np.take_along_axis(s_ref, got, axis=1)
    assert np.all(sel[:, :-1] >= sel[:, 1:] - tau)
    return int((~safe).sum())


@pytest.mark.parametrize("T,d,E,K,act,rw", [
    (512, 128, 8, 2, torch.float32, torch.float32),
    (1000, 2048, 128, 8, torch.bfloat16, torch.float32),
    (257, 2048, 128, 8, torch.bfloat16, torch.bfloat16),
    (130, 72, 300, 7, torch.bfloat16, torch.float32),
])
def test_capture_random_data(r3, T, d, E, K, act, rw):
    x = torch.randn(T, d).to(act)
    w = (torch.randn(E, d) * 0.02).to(rw)
    s = r3.make_shape(T, d, E, K, 8, act=act, router=rw, idx=idx_dtype(E))
    idx, logits = r3.capture_topk(s, x.cuda(), w.cuda(), want_logits=True)
    ref_s = O.router_logits(f64(x), f64(w))
    assert rel_err(logits.cpu().numpy(), ref_s) < TOL_F32
    check_record_against_logits(idx.cpu().numpy(), ref_s, K)
    only_idx, none = r3.capture_topk(s, x.cuda(), w.cuda())
    assert none is None and torch.equal(only_idx, idx)


def test_capture_batched_layers(r3):
    L, T, d, E, K = 5, 70, 256, 128, 8
    x = torch.randn(L, T, d).to(torch.bfloat16)
    w = (torch.randn(L, E, d) * 0.02).to(torch.bfloat16)
    s = r3.make_shape(T, d, E, K, 8, router=torch.bfloat16)
    idx, logits = r3.capture_topk_batched(s, L, x.cuda(), w.cuda(), want_logits=True)
    for l in range(L):
        ref_s = O.router_logits(f64(x[l]), f64(w[l]))
        assert rel_err(logits[l].cpu().numpy(), ref_s) < TOL_F32
        check_record_against_logits(idx[l].cpu().numpy(), ref_s, K)


@pytest.mark.parametrize("L,T,d,E,K,rw", [
    (50, 70, 256, 128, 8, torch.bfloat16),       # fewer tokens than one CTA of the pair holds
    (60, 130, 320, 48, 3, torch.float32),        # two tokens for the second CTA, three weight planes
    (50, 100, 256, 256, 8, torch.bfloat16),      # 256 experts: two column chunks per thread, int16 record
    (47, 256, 512, 64, 1, torch.float32),        # a full tile, K = 1
])
def test_capture_batched_layers_pair_form(r3, L, T, d, E, K, rw):
    """46 to 74 one-tile layers in a launch: the range in which the router kernel gives every tile a
    pair of CTAs with the tokens on the M side of the MMA (the 48-layer decode batch of the paper's
    setting is the full-size case).  Small-integer data, so logits and record must equal the
    oracle's bit for bit; every token of layer 1 is a planted tie (experts 2, 5 and 17 share their
    weights), which sends those tokens through the exact second selection, and layer 2 holds the
    signed zeros."""
    rng = np.random.default_rng(L + T + E)
    x = torch.from_numpy(rng.integers(-3, 4, (L, T, d)).astype(np.float32)).to(torch.bfloat16)
    w = torch.from_numpy(rng.integers(-2, 3, (L, E, d)).astype(np.float32)).to(rw)
    w[1, 5] = w[1, 2]
    w[1, 17] = w[1, 2]
    w[1, E - 1] = w[1, 0]
    plant_signed_zeros(x[2], w[2])
    s = r3.make_shape(T, d, E, K, 8, router=rw, idx=idx_dtype(E))
    idx, logits = r3.capture_topk_ws(s, L, x.cuda(), w.cuda(), want_logits=True)
    for l in range(L):
        ref_s = O.router_logits(f64(x[l]), f64(w[l]))
        assert np.array_equal(logits[l].cpu().numpy().astype(np.float64), ref_s), l
        assert np.array_equal(idx[l].cpu().numpy().astype(np.int64), O.topk_indices(ref_s, K)), l
    only_idx, none = r3.capture_topk_ws(s, L, x.cuda(), w.cuda())
    assert none is None and torch.equal(only_idx, idx)
    _, only_logits = r3.capture_topk_ws(s, L, x.cuda(), w.cuda(), want_idx=False, want_logits=True)
    assert torch.equal(only_logits, logits)


# ------------------------------------------------------------------ grouped SwiGLU experts
def run_swiglu_case(r3, T, d, E, K, F, act, tol, seed=0):
    rng = np.random.default_rng(seed + T)
    pop = rng.random(E) ** 2 + 0.01
    keys = rng.random((T, E)) * pop[None, :]
    idx_np = np.argsort(-keys, axis=1)[:, :K]
    _, offsets, ros, sor = O.permutation(idx_np, E)
    x = torch.randn(T, d).to(act)
    wg = (torch.randn(E, F, d) * 0.05).to(act)
    wu = (torch.randn(E, F, d) * 0.05).to(act)
    wd = (torch.randn(E, d, F) * 0.05).to(act)
    xp = x[torch.from_numpy(sor.astype(np.int64)) // K].contiguous()
    s = r3.make_shape(T, d, E, K, F, act=act)
    st = r3.new_status("cuda")
    o = r3.grouped_swiglu(s, xp.cuda(), torch.from_numpy(offsets).cuda(), wg.cuda(), wu.cuda(),
                          wd.cuda(), dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    eo = O.expert_outputs(f64(x), idx_np, f32(wg), f32(wu), f32(wd))     # [T, K, d]
    ref = np.empty((T * K, d))
    ref[ros.reshape(-1).astype(np.int64)] = eo.reshape(T * K, d)
    err = rel_err(f64(o), ref)
    assert err < tol, err
    o2 = r3.grouped_swiglu(s, xp.cuda(), torch.from_numpy(offsets).cuda(), wg.cuda(), wu.cuda(),
                           wd.cuda())
    assert torch.equal(o, o2)
    if act == torch.bfloat16:
        # the gather form reads the same rows in place from x: bit-identical
        st2 = r3.new_status("cuda")
        o3 = r3.grouped_swiglu_gather(s, x.cuda(), torch.from_numpy(sor.astype(np.int32)).cuda(),
                                      torch.from_numpy(offsets).cuda(), wg.cuda(), wu.cuda(),
                                      wd.cuda(), dev_status=st2)
        assert st2.item() == 0
        assert torch.equal(o, o3)


@pytest.mark.parametrize("T,d,E,K,F", [(64, 128, 8, 2, 256), (300, 72, 5, 3, 40), (7, 8, 3, 1, 8)])
def test_grouped_swiglu_f32(r3, T, d, E, K, F):
    run_swiglu_case(r3, T, d, E, K, F, torch.float32, TOL_F32)


@pytest.mark.parametrize("T,d,E,K,F", [
    (256, 256, 4, 2, 128),        # a few full tiles
    (300, 2048, 16, 8, 768),      # the paper-like layer shape, ragged expert sizes
    (77, 136, 6, 3, 72),          # ragged d, F (k and n tails), experts smaller than a tile
    (1500, 512, 3, 2, 264),       # experts spanning many row tiles
])
def test_grouped_swiglu_bf16_tensor_cores(r3, T, d, E, K, F):
    run_swiglu_case(r3, T, d, E, K, F, torch.bfloat16, TOL_BF16)


def test_expert_down_twice_from_one_work_list(r3):
    """The down projection reads the work list the up projection left in the workspace.  Its
    clusters claim items from a counter in that list; the launch re-arms the counter when it
    ends, so a second launch from the same list computes every item again.  T and E are chosen
    so that the list holds several times as many items as there are clusters (most of them are
    claimed from the counter, not taken by position)."""
    T, d, E, K, F = 6000, 1024, 24, 4, 264
    act = torch.bfloat16
    rng = np.random.default_rng(5)
    idx_np = np.argsort(-rng.random((T, E)), axis=1)[:, :K]
    _, offsets, ros, sor = O.permutation(idx_np, E)
    x = torch.randn(T, d).to(act)
    wg = (torch.randn(E, F, d) * 0.05).to(act).cuda()
    wu = (torch.randn(E, F, d) * 0.05).to(act).cuda()
    wd = (torch.randn(E, d, F) * 0.05).to(act).cuda()
    xp = x[torch.from_numpy(sor.astype(np.int64)) // K].contiguous().cuda()
    off = torch.from_numpy(offsets).cuda()
    s = r3.make_shape(T, d, E, K, F, act=act)
    st = r3.new_status("cuda")
    whole = r3.grouped_swiglu(s, xp, off, wg, wu, wd, dev_status=st)
    ws = r3.workspace(r3.grouped_swiglu_workspace_bytes(s), "cuda")
    r3.expert_up_swiglu(s, xp, off, wg, wu, ws, dev_status=st)
    o1 = torch.full((T * K, d), float("nan"), dtype=act, device="cuda")
    o2 = torch.full((T * K, d), float("nan"), dtype=act, device="cuda")
    r3.expert_down(s, wd, o1, ws, dev_status=st)
    r3.expert_down(s, wd, o2, ws, dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert torch.equal(o1, whole)
    assert torch.equal(o2, whole)
