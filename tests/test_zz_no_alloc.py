"""r3_permute_static: the dispatch step for callers that cannot allocate device memory where
they call from (their device memory belongs to another component's pool, or their step has a
fixed memory plan).  Its scratch is a fixed array inside the library, so the check is simply that
it gives r3_permute's results (and the oracle's grouping) bit for bit - twice in a row, since
every call reuses the same array and finds the previous call's contents in it - and that it
refuses problems that do not fit the array.  Collected last on purpose (file name), so that a run that stops at the first
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
    from oracle import r3_oracle as O
    from paper_2510_11370_b200 import r3
    # Two different problems back to back, BOTH with more than 16 chunks of 256 tokens, so both
    # take the kernels that keep their [expert][chunk] counters in the library's array (a smaller
    # batch is dispatched by one cluster out of shared memory and never touches it).  The first
    # fills 300 x 36 counters; the second lays its 64 x 20 over the first one's leftovers and must
    # not be affected by them.
    for seed, (T, E, K, d) in enumerate([(9000, 300, 4, 64), (5000, 64, 8, 256)]):
        assert (T + 255) // 256 > 16
        idx, x = make_inputs(seed, T, E, K, d)
        s = r3.make_shape(T, d, E, K, 8, idx=idx.dtype)
        want = r3.permute(s, idx, x)
        out = empty_outputs(T, E, K, d)
        st = r3.new_status("cuda")
        torch.cuda.synchronize()
        requests = torch.cuda.memory_stats()["allocation.all.allocated"]
        got = r3.permute_static(s, idx, x, *out, dev_status=st)
        torch.cuda.synchronize()
        # the caller's allocator was asked for nothing during the call
        assert torch.cuda.memory_stats()["allocation.all.allocated"] == requests
        assert st.item() == 0
        for a, b in zip(got, want):
            assert torch.equal(a, b)              # integer maps and copied rows: bit-exact
        # and against the oracle's stable grouping, not only against the library's other entry
        counts, offsets, ros, sor = O.permutation(idx.cpu().to(torch.int64).numpy(), E)
        for a, b in zip(got[:4], (counts, offsets, ros, sor)):
            assert np.array_equal(a.cpu().numpy(), b)
        assert torch.equal(got[4].cpu(), x.cpu()[torch.from_numpy(sor.astype(np.int64)) // K])


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
