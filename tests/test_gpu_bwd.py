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
