"""r3_permute_static: the dispatch step for callers that cannot allocate device memory where
they call from (their device memory belongs to another component's pool, or their step has a
fixed memory plan).  Its scratch is a fixed array inside the library, so the check is simply that
it gives r3_permute's results bit for bit - twice in a row, since every call reuses the same
array and finds the previous call's contents in it - and that it refuses problems that do not
fit the array.  Collected last on purpose (file name), so that a run that stops at the first
failure has already run every other test."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


def make_inputs(seed, T, E, K, d):
    rng = np.random.default_rng(seed)
    pop = rng.random(E) ** 3 + 1e-3
    idx = np.argsort(-(rng.random((T, E)) * pop[None, :]), axis=1)[:, :K]
    dtype = torch.uint8 if E <= 256 else torch.int16
    x = torch.from_numpy(rng.standard_normal((T, d)).astype(np.float32)).to(torch.bfloat16)
    return torch.from_numpy(idx).to(dtype).cuda(), x.cuda()


def empty_outputs(T, E, K, d):
    dev = "cuda"
    return (torch.full((E,), -7, dtype=torch.int32, device=dev),
            torch.full((E + 1,), -7, dtype=torch.int32, device=dev),
            torch.full((T, K), -7, dtype=torch.int32, device=dev),
            torch.full((T * K,), -7, dtype=torch.int32, device=dev),
            torch.zeros((T * K, d), dtype=torch.bfloat16, device=dev))


def test_permute_static_matches_permute_on_two_calls_in_a_row():
    from paper_2510_11370_b200 import r3
    # two different problems back to back: the second call finds the first one's counters in the
    # shared scratch (more chunks and more experts first, then fewer) and must not be affected
    for seed, (T, E, K, d) in enumerate([(5000, 300, 4, 64), (1111, 128, 8, 256)]):
        idx, x = make_inputs(seed, T, E, K, d)
        s = r3.make_shape(T, d, E, K, 8, idx=idx.dtype)
        want = r3.permute(s, idx, x)
        out = empty_outputs(T, E, K, d)
        st = r3.new_status("cuda")
        got = r3.permute_static(s, idx, x, *out, dev_status=st)
        torch.cuda.synchronize()
        assert st.item() == 0
        for a, b in zip(got, want):
            assert torch.equal(a, b)              # integer maps and copied rows: bit-exact


def test_permute_static_refuses_what_does_not_fit_its_scratch():
    from paper_2510_11370_b200 import r3
    T, E, K = 256 * 300, 1000, 2                  # 1000 experts x 300 chunks > 262144 counters
    s = r3.make_shape(T, 8, E, K, 8, idx=torch.int16)
    idx = torch.zeros((T, K), dtype=torch.int16, device="cuda")
    out = empty_outputs(T, E, K, 8)
    with pytest.raises(r3.R3Error) as err:
        r3.permute_static(s, idx, None, *out[:4], None)
    assert err.value.code == r3.R3_ERR_SCRATCH_LIMIT
    assert "262144" in str(err.value)
    assert all(int(t.flatten()[0]) == -7 for t in out[:4])    # nothing was launched
