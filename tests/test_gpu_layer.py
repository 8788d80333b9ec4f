"""Whole replayed layer (forward + router-logit backward) through the C ABI against the oracle,
on the benchmark configurations.  Small configurations are compared element by element; the
large ones compare all integer work and the gates exactly/fully, and the expert-dependent
outputs on sampled tokens that the oracle evaluates one by one."""
import copy

import numpy as np
import pytest
import torch

from oracle import r3_oracle as O
from paper_2510_11370_b200 import synth
from tests.helpers import Case, f32, f64, rel_err
from tests.test_gpu_kernels import check_record_against_logits

pytestmark = pytest.mark.gpu

TOL_BF16 = 2e-2
TOL_F32 = 1e-5


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import r3 as mod
    return mod


def run_layer(r3, case, stepwise=False):
    s = r3.shape_of(case.w)
    c = case.cuda()
    st = r3.new_status("cuda")
    if not stepwise:
        y, ds, g = r3.replay_layer(s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"],
                                   c["w_down"], c["dy"], dev_status=st)
        torch.cuda.synchronize()
        assert st.item() == 0
        return dict(y=y, ds=ds, g=g)
    _, logits = r3.capture_topk_ws(s, 1, c["x"], c["w_r"], want_idx=False, want_logits=True)
    g = r3.replay_gate_fwd(s, logits, c["idx"], dev_status=st)
    counts, offsets, ros, sor, xp = r3.permute(s, c["idx"], c["x"], dev_status=st)
    o = r3.grouped_swiglu(s, xp, offsets, c["w_gate"], c["w_up"], c["w_down"], dev_status=st)
    y = r3.combine(s, o, ros, g)
    dg = r3.combine_bwd_gates(s, c["dy"], o, ros)
    ds = r3.replay_gate_bwd(s, g, dg, c["idx"])
    torch.cuda.synchronize()
    assert st.item() == 0
    return dict(y=y, ds=ds, g=g, logits=logits, counts=counts, offsets=offsets, ros=ros, sor=sor,
                xp=xp, o=o, dg=dg)


def check_full(case, got, ref, tol):
    assert rel_err(f64(got["g"]), ref["g"]) < max(tol * 1e-2, 1e-5)
    assert rel_err(f64(got["y"]), ref["y"]) < tol
    assert rel_err(f64(got["ds"]), ref["ds"]) < tol
    if "sor" in got:
        counts, offsets, ros, sor = O.permutation(case.idx_np(), case.w.E)
        assert np.array_equal(got["counts"].cpu().numpy(), counts)
        assert np.array_equal(got["offsets"].cpu().numpy(), offsets)
        assert np.array_equal(got["ros"].cpu().numpy(), ros)
        assert np.array_equal(got["sor"].cpu().numpy(), sor)
        assert torch.equal(got["xp"].cpu(), case.x[torch.from_numpy(sor.astype(np.int64)) // case.w.K])
        assert rel_err(got["logits"].cpu().numpy(), ref["s"]) < 1e-5
        assert rel_err(f64(got["dg"]), ref["dg"]) < tol


def test_config1_tiny_fp32_layer(r3):
    case = Case(synth.WORKLOADS["c1_tiny_fp32"])
    own = O.topk_indices(case.s, 2)
    differs = (np.sort(own, axis=1) != np.sort(case.idx_np(), axis=1)).any(axis=1).mean()
    assert 0.04 < differs < 0.2                        # about 10% of tokens replay another expert
    ref = case.oracle_layer()
    check_full(case, run_layer(r3, case, stepwise=True), ref, TOL_F32)
    check_full(case, run_layer(r3, case), ref, TOL_F32)


def test_config1_replay_of_own_topk_is_the_ordinary_layer(r3):
    """Replaying the record that the library's own capture kernel makes from the training logits
    reproduces the ordinary MoE layer (Eqs. train_gate / train_output)."""
    w = synth.WORKLOADS["c1_tiny_fp32"]
    case = Case(w)
    s = r3.shape_of(w)
    c = case.cuda()
    own, _ = r3.capture_topk(s, c["x"], c["w_r"])
    assert np.array_equal(own.cpu().numpy().astype(np.int64), O.topk_indices(case.s, w.K))
    y, _, _ = r3.replay_layer(s, c["x"], c["w_r"], own, c["w_gate"], c["w_up"], c["w_down"],
                              c["dy"])
    y_ref = O.train_output(f64(case.x), f64(case.w_r), w.K, f64(case.w_gate), f64(case.w_up),
                           f64(case.w_down))
    assert rel_err(f64(y), y_ref) < TOL_F32


def test_config2_bf16_layer_full(r3):
    case = Case(synth.WORKLOADS["c2_layer_bf16"])
    ref = case.oracle_layer()
    check_full(case, run_layer(r3, case, stepwise=True), ref, TOL_BF16)
    got = run_layer(r3, case)
    check_full(case, got, ref, TOL_BF16)
    again = run_layer(r3, case)
    assert torch.equal(got["y"], again["y"]) and torch.equal(got["ds"], again["ds"])


def sampled_check(case, got, n_samples, tol, seed=0):
    """Sampled tokens through the oracle's layer (every token's result depends on that token
    alone, so the oracle is run on the sampled rows as a batch of their own): y and dlogits of
    those tokens, and - when the run kept them - the expert outputs o of their K rows."""
    w = case.w
    rng = np.random.default_rng(seed)
    sel = np.sort(rng.choice(w.T, size=n_samples, replace=False))
    ref = O.layer_fwd_bwd(f64(case.x[sel]), f64(case.w_r), case.idx_np()[sel], case.w_gate,
                          case.w_up, case.w_down, f64(case.dy[sel]))
    tsel = torch.from_numpy(sel)
    err_y = rel_err(f64(got["y"].cpu()[tsel]), ref["y"])
    err_ds = rel_err(f64(got["ds"].cpu()[tsel]), ref["ds"])
    assert err_y < tol and err_ds < tol, (err_y, err_ds)
    errs = dict(y=err_y, ds=err_ds)
    if "o" in got:
        rows = got["ros"].cpu()[tsel].to(torch.int64)                 # [n, K] grouped rows
        o_rows = f64(got["o"].cpu()[rows.reshape(-1)]).reshape(n_samples, w.K, w.d)
        errs["o"] = rel_err(o_rows, ref["eo"])
        assert errs["o"] < tol, errs
    return errs


def expert_rows_check(case, got, experts, tol):
    """ALL rows of the given experts: o[offsets[e] : offsets[e+1]] against the oracle's expert
    network on the rows the oracle's own dispatch gives that expert (the dispatch itself is
    compared bit for bit elsewhere in the same test).  Returns {expert: (rows, error)}."""
    w = case.w
    _, offsets, _, sor = O.permutation(case.idx_np(), w.E)
    o = got["o"]
    out = {}
    for e in experts:
        lo, hi = int(offsets[e]), int(offsets[e + 1])
        if hi == lo:
            out[int(e)] = (0, 0.0)
            continue
        tokens = torch.from_numpy(sor[lo:hi].astype(np.int64) // w.K)
        ref = O.swiglu_expert(f64(case.x[tokens]), case.w_gate[e], case.w_up[e], case.w_down[e])
        err = rel_err(f64(o[lo:hi].cpu()), ref)
        assert err < tol, (int(e), hi - lo, err)
        out[int(e)] = (hi - lo, err)
    return out


def pick_experts(counts):
    """Experts whose row counts exercise the tile schedule: the largest, one just over one
    256-row tile (closest to 257..272), one whose count is not a multiple of 16, the smallest
    non-empty one, and every empty one's two neighbours."""
    counts = np.asarray(counts)
    chosen = [int(np.argmax(counts))]
    over = np.where(counts > 256)[0]
    if over.size:
        chosen.append(int(over[np.argmin(np.abs(counts[over] - 264))]))
    ragged = np.where((counts % 16 != 0) & (counts > 0))[0]
    if ragged.size:
        chosen.append(int(ragged[np.argmin(counts[ragged])]))          # the smallest ragged one
        chosen.append(int(ragged[np.argmax(counts[ragged] % 16)]))
    nonempty = np.where(counts > 0)[0]
    chosen.append(int(nonempty[np.argmin(counts[nonempty])]))
    for e in np.where(counts == 0)[0]:
        chosen += [int(x) for x in (e - 1, e + 1) if 0 <= x < counts.size and counts[x] > 0]
    seen, out = set(), []
    for e in chosen:
        if e not in seen:
            seen.add(e)
            out.append(e)
    return out


class LazyWeights:
    """Per-expert float64 view of a stored [E, ...] weight tensor (converted on access)."""

    def __init__(self, t):
        self.t = t

    def __len__(self):
        return self.t.shape[0]

    def __getitem__(self, i):
        return self.t[int(i)].to(torch.float64).numpy()


def big_case(w):
    case = Case(w, device="cuda")
    case.w_gate, case.w_up, case.w_down = (LazyWeights(t) for t in
                                           (case.w_gate, case.w_up, case.w_down))
    return case


def run_big(r3, case, raw):
    s = r3.shape_of(case.w)
    st = r3.new_status("cuda")
    c = {k: getattr(case, k).cuda() for k in ("x", "dy", "w_r", "idx")}
    wg, wu, wd = (t.cuda() for t in raw)
    _, logits = r3.capture_topk_ws(s, 1, c["x"], c["w_r"], want_idx=False, want_logits=True)
    g = r3.replay_gate_fwd(s, logits, c["idx"], dev_status=st)
    counts, offsets, ros, sor, xp = r3.permute(s, c["idx"], c["x"], dev_status=st)
    o = r3.grouped_swiglu(s, xp, offsets, wg, wu, wd, dev_status=st)
    y = r3.combine(s, o, ros, g)
    dg = r3.combine_bwd_gates(s, c["dy"], o, ros)
    ds = r3.replay_gate_bwd(s, g, dg, c["idx"])
    y2, ds2, g2 = r3.replay_layer(s, c["x"], c["w_r"], c["idx"], wg, wu, wd, c["dy"],
                                  dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    # the one-pass finish of the layer sums the gate gradient in another (fixed) order than
    # r3_combine_bwd_gates: y and the gates agree bit for bit, dlogits to float32 rounding
    assert torch.equal(y, y2) and torch.equal(g, g2)
    assert (ds - ds2).abs().max().item() <= 1e-5 * ds.abs().max().item()
    return dict(y=y, ds=ds, g=g, logits=logits, counts=counts, offsets=offsets, ros=ros, sor=sor,
                xp=xp, o=o)


def check_big(case, got, tol, n_samples=256):
    w = case.w
    counts, offsets, ros, sor = O.permutation(case.idx_np(), w.E)
    assert np.array_equal(got["counts"].cpu().numpy(), counts)
    assert np.array_equal(got["offsets"].cpu().numpy(), offsets)
    assert np.array_equal(got["ros"].cpu().numpy(), ros)
    assert np.array_equal(got["sor"].cpu().numpy(), sor)
    assert torch.equal(got["xp"].cpu(), case.x[torch.from_numpy(sor.astype(np.int64)) // w.K])
    assert rel_err(got["logits"].cpu().numpy(), case.s) < 1e-5
    assert rel_err(f64(got["g"]), O.replay_gate(case.s, case.idx_np())) < 1e-5
    errs = sampled_check(case, got, n_samples, tol)
    rows = expert_rows_check(case, got, pick_experts(counts), tol)
    print(f"{w.name}: {n_samples} sampled tokens {errs}; all rows of experts "
          f"{ {e: (n, round(err, 5)) for e, (n, err) in rows.items()} }")
    return counts


def test_config3_skewed_routing_full_size(r3):
    w = synth.WORKLOADS["c3_skewed"]
    case = Case(w, device="cuda")
    raw = (case.w_gate, case.w_up, case.w_down)
    case.w_gate, case.w_up, case.w_down = (LazyWeights(t) for t in raw)
    got = run_big(r3, case, raw)
    counts = check_big(case, got, TOL_BF16)
    # the Zipf bias really skews the load: a few experts take most rows, some take (almost) none
    assert counts.max() > 20 * max(1, np.median(counts)) or counts.max() > w.T // 2
    assert counts.min() < w.T * w.K // w.E // 4
    # the largest expert spans over a hundred 256-row token tiles, and ragged tails exist
    assert counts.max() > 100 * 256 and np.any(counts % 16 != 0)


def test_config4_capture_then_replay_round_trip(r3):
    # inference side: 48 layers x 256 decode tokens, bf16 router, uint8 record, one launch
    wc = synth.WORKLOADS["c4_capture"]
    L = wc.layers
    xs = torch.stack([synth.activations(wc, "cpu", l) for l in range(L)])
    wr = torch.stack([synth.router_weight(wc, "cpu", l) for l in range(L)])
    s = r3.shape_of(wc)
    rec, logits = r3.capture_topk_batched(s, L, xs.cuda(), wr.cuda(), want_logits=True)
    assert rec.dtype == torch.uint8 and rec.shape == (L, wc.T, wc.K)
    near = 0
    for l in range(L):
        ref_s = O.router_logits(f64(xs[l]), f64(wr[l]))
        assert rel_err(logits[l].cpu().numpy(), ref_s) < 1e-5
        near += check_record_against_logits(rec[l].cpu().numpy(), ref_s, wc.K)
    assert near < 0.05 * L * wc.T

    # training side: a recorded 65536-token batch replayed through one layer.  The record is the
    # library's own capture of that batch; the oracle works from its own TopKMask of the same
    # inputs, and parity is judged on the tokens where the two records agree bit for bit.
    wr_ = synth.WORKLOADS["c4_replay"]
    case = Case(synth.scaled(wr_, record="noise", sigma=0.0), device="cuda")
    raw = (case.w_gate, case.w_up, case.w_down)
    case.w_gate, case.w_up, case.w_down = (LazyWeights(t) for t in raw)
    s2 = r3.shape_of(wr_)
    xg, wrg = case.x.cuda(), case.w_r.cuda()
    gpu_rec, _ = r3.capture_topk(s2, xg, wrg)
    oracle_rec = O.topk_indices(case.s, wr_.K)
    check_record_against_logits(gpu_rec.cpu().numpy(), case.s, wr_.K)
    same = (gpu_rec.cpu().numpy().astype(np.int64) == oracle_rec).all(axis=1)
    assert same.mean() > 0.95
    st = r3.new_status("cuda")
    y, ds, g = r3.replay_layer(s2, xg, wrg, gpu_rec, *(t.cuda() for t in raw), case.dy.cuda(),
                               dev_status=st)
    torch.cuda.synchronize()
    assert st.item() == 0
    assert np.allclose(g.cpu().numpy().sum(axis=1), 1.0, atol=1e-5)
    rng = np.random.default_rng(1)
    sel = np.sort(rng.choice(np.nonzero(same)[0], size=256, replace=False))
    ref = O.layer_fwd_bwd(f64(case.x[sel]), f64(case.w_r), oracle_rec[sel], case.w_gate,
                          case.w_up, case.w_down, f64(case.dy[sel]))
    tsel = torch.from_numpy(sel)
    err_y, err_ds = rel_err(f64(y.cpu()[tsel]), ref["y"]), rel_err(f64(ds.cpu()[tsel]), ref["ds"])
    print(f"c4 round trip: 256 sampled tokens y {err_y:.2e} dlogits {err_ds:.2e}")
    assert err_y < TOL_BF16 and err_ds < TOL_BF16
    del y, ds, g

    # the same batch replayed from the ORACLE's record (an input that does not come from the
    # library): dispatch bit for bit, all rows of chosen experts, 256 sampled tokens
    case.idx = torch.from_numpy(oracle_rec).to(torch.uint8)
    got = run_big(r3, case, raw)
    check_big(case, got, TOL_BF16)


def test_host_buffer_layer_and_two_batches_in_flight(r3):
    """r3_replay_layer_host gives the device path's bits, and r3_replay_layer_host_enqueue with two
    batches in flight (own stream, workspace and pinned buffers each) gives, for each batch, the
    bits of running it alone."""
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], T=1000)
    cases = [Case(w, device="cuda")]
    cases.append(copy.copy(cases[0]))
    cases[1].x = cases[1].x.flip(0).contiguous()          # a second batch with other rows
    cases[1].dy = cases[1].dy.flip(0).contiguous()
    cases[1].idx = cases[1].idx.flip(0).contiguous()
    s = r3.shape_of(w)
    st = r3.new_status("cuda")
    dev = {k: getattr(cases[0], k).cuda() for k in ("w_r", "w_gate", "w_up", "w_down")}
    alone, bufs = [], []
    for c in cases:
        y, ds, _ = r3.replay_layer(s, c.x.cuda(), dev["w_r"], c.idx.cuda(), dev["w_gate"],
                                   dev["w_up"], dev["w_down"], c.dy.cuda(), dev_status=st)
        torch.cuda.synchronize()
        alone.append((y.cpu(), ds.cpu()))
        bufs.append(dict(x=c.x.pin_memory(), dy=c.dy.pin_memory(), idx=c.idx.pin_memory(),
                         y=torch.empty((w.T, w.d), dtype=c.x.dtype).pin_memory(),
                         ds=torch.empty((w.T, w.E), dtype=torch.float32).pin_memory(),
                         ws=r3.workspace(r3.replay_layer_host_workspace_bytes(s), "cuda"),
                         stream=torch.cuda.Stream()))
    b = bufs[0]
    r3.replay_layer_host(s, b["x"], dev["w_r"], b["idx"], dev["w_gate"], dev["w_up"], dev["w_down"],
                         b["dy"], b["y"], b["ds"], ws=b["ws"], dev_status=st)
    assert torch.equal(b["y"], alone[0][0]) and torch.equal(b["ds"], alone[0][1])
    for rounds in range(3):
        for b in bufs:
            b["y"].zero_()
            b["ds"].zero_()
        for b in bufs:
            r3.replay_layer_host_enqueue(s, b["x"], dev["w_r"], b["idx"], dev["w_gate"],
                                         dev["w_up"], dev["w_down"], b["dy"], b["y"], b["ds"],
                                         ws=b["ws"], dev_status=st, stream=b["stream"])
        for b in bufs:
            b["stream"].synchronize()
        for b, (y, ds) in zip(bufs, alone):
            assert torch.equal(b["y"], y) and torch.equal(b["ds"], ds)
    assert st.item() == 0


def test_host_buffer_layer_in_token_chunks(r3):
    """From 16384 tokens on r3_replay_layer_host sends the batch through in chunks of tokens
    (copies of one chunk beside the compute of another).  Every step of the layer is per token, so
    a chunk must come out with the bits of running it alone on the device path (the whole batch
    in one launch may differ in the last bits: the router kernel splits d differently for another
    token count, so that run is compared within a bf16 rounding step); two such calls in flight
    on streams of their own must not disturb each other."""
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], T=40000, d=256, E=16, K=4, F=136)
    cases = [Case(w, device="cuda")]
    cases.append(copy.copy(cases[0]))
    cases[1].x = cases[1].x.flip(0).contiguous()
    cases[1].dy = cases[1].dy.flip(0).contiguous()
    cases[1].idx = cases[1].idx.flip(0).contiguous()
    s = r3.shape_of(w)
    starts = r3.replay_layer_host_chunks(s)
    assert starts == [0, 8192, 16384, 24576, 32768, 36352, 38144, 40000]
    st = r3.new_status("cuda")
    dev = {k: getattr(cases[0], k).cuda() for k in ("w_r", "w_gate", "w_up", "w_down")}
    alone, bufs = [], []
    for c in cases:
        ys, dss = [], []
        for t0, t1 in zip(starts, starts[1:]):
            n = t1 - t0
            sp = r3.shape_of(synth.scaled(w, T=n))
            y, ds, _ = r3.replay_layer(sp, c.x[t0:t0 + n].cuda(), dev["w_r"],
                                       c.idx[t0:t0 + n].cuda(), dev["w_gate"], dev["w_up"],
                                       dev["w_down"], c.dy[t0:t0 + n].cuda(), dev_status=st)
            torch.cuda.synchronize()
            ys.append(y.cpu())
            dss.append(ds.cpu())
        alone.append((torch.cat(ys), torch.cat(dss)))
        bufs.append(dict(x=c.x.pin_memory(), dy=c.dy.pin_memory(), idx=c.idx.pin_memory(),
                         y=torch.empty((w.T, w.d), dtype=c.x.dtype).pin_memory(),
                         ds=torch.empty((w.T, w.E), dtype=torch.float32).pin_memory(),
                         ws=r3.workspace(r3.replay_layer_host_workspace_bytes(s), "cuda"),
                         stream=torch.cuda.Stream()))
    c = cases[0]
    y_whole, ds_whole, _ = r3.replay_layer(s, c.x.cuda(), dev["w_r"], c.idx.cuda(), dev["w_gate"],
                                           dev["w_up"], dev["w_down"], c.dy.cuda(), dev_status=st)
    b = bufs[0]
    r3.replay_layer_host(s, b["x"], dev["w_r"], b["idx"], dev["w_gate"], dev["w_up"], dev["w_down"],
                         b["dy"], b["y"], b["ds"], ws=b["ws"], dev_status=st)
    assert torch.equal(b["y"], alone[0][0]) and torch.equal(b["ds"], alone[0][1])
    assert rel_err(f64(b["y"]), f64(y_whole)) < 2.0 ** -7
    assert rel_err(f64(b["ds"]), f64(ds_whole)) < 1e-4
    for rounds in range(2):
        for b in bufs:
            b["y"].zero_()
            b["ds"].zero_()
        for b in bufs:
            r3.replay_layer_host_enqueue(s, b["x"], dev["w_r"], b["idx"], dev["w_gate"],
                                         dev["w_up"], dev["w_down"], b["dy"], b["y"], b["ds"],
                                         ws=b["ws"], dev_status=st, stream=b["stream"])
        for b in bufs:
            b["stream"].synchronize()
        for b, (y, ds) in zip(bufs, alone):
            assert torch.equal(b["y"], y) and torch.equal(b["ds"], ds)
    assert st.item() == 0


@pytest.mark.parametrize("name,T", [("c1_tiny_fp32", 512), ("c2_layer_bf16", 1500)])
def test_second_pass_over_the_same_record(r3, name, T):
    """r3_replay_layer_same_record uses the dispatch and the work lists that r3_replay_layer left
    in the workspace: with new activations, new upstream gradient and scaled weights (the Update
    stage after the Recompute stage) it gives the bits of a fresh r3_replay_layer call."""
    w = synth.scaled(synth.WORKLOADS[name], T=T)
    case = Case(w, device="cuda")
    s = r3.shape_of(w)
    c = case.cuda()
    st = r3.new_status("cuda")
    ws = r3.workspace(r3.replay_layer_workspace_bytes(s), "cuda")
    first = r3.replay_layer(s, c["x"], c["w_r"], c["idx"], c["w_gate"], c["w_up"], c["w_down"],
                            c["dy"], ws=ws, dev_status=st)
    x2 = (c["x"].flip(1) * 0.5).contiguous()
    dy2 = c["dy"].flip(0).contiguous()
    wd2 = (c["w_down"] * 1.25).contiguous()
    for _ in range(2):
        again = r3.replay_layer_same_record(s, x2, c["w_r"], c["idx"], c["w_gate"], c["w_up"], wd2,
                                            dy2, ws=ws, dev_status=st)
        torch.cuda.synchronize()
        fresh = r3.replay_layer(s, x2, c["w_r"], c["idx"], c["w_gate"], c["w_up"], wd2, dy2,
                                dev_status=st)
        torch.cuda.synchronize()
        for a, b in zip(again, fresh):
            assert torch.equal(a, b)
    assert st.item() == 0
    assert not torch.equal(first[0], again[0])
