"""The C-ABI library loads, exports every symbol the header declares, and rejects bad arguments
on the host (no kernel is launched by anything in this file)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def r3():
    from paper_2510_11370_b200 import build
    build.build()
    from paper_2510_11370_b200 import r3 as mod
    return mod


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "r3.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(r3_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound(r3):
    syms = declared_symbols()
    assert len(syms) >= 15
    for name in syms:
        assert hasattr(r3.lib, name), name
    assert sorted(r3.EXPORTS) == syms


def test_status_strings(r3):
    for code in range(5):
        s = r3.lib.r3_status_string(code).decode()
        assert s and (code == 0) == (s == "R3_OK")
    assert "unknown" in r3.lib.r3_status_string(99).decode()


def test_shape_struct_matches_header_layout(r3):
    assert ctypes.sizeof(r3.Shape) == 32
    assert [f[0] for f in r3.Shape._fields_] == ["T", "d", "E", "K", "F", "act_dtype",
                                                  "router_w_dtype", "idx_type"]


@pytest.mark.parametrize("kw", [
    dict(K=9, E=8),                    # K > E
    dict(E=300),                       # uint8 record cannot hold 300 experts
    dict(d=100),                       # d not a multiple of 8
    dict(T=-1),
    dict(F=0),
])
def test_bad_shapes_are_rejected_on_the_host(r3, kw):
    base = dict(T=16, d=64, E=8, K=2, F=64)
    base.update(kw)
    s = r3.make_shape(**base)
    assert r3.lib.r3_replay_gate_fwd(ctypes.byref(s), None, None, None, None, None) == 1
    assert r3.lib.r3_combine(ctypes.byref(s), None, None, None, None, None) == 1
    assert r3.permute_workspace_bytes(s) == 0
    assert r3.replay_layer_workspace_bytes(s) == 0


def test_null_pointers_and_workspace_errors(r3):
    s = r3.make_shape(16, 64, 8, 2, 64)
    assert r3.lib.r3_replay_gate_fwd(ctypes.byref(s), None, None, None, None, None) == 1
    assert r3.lib.r3_capture_topk(ctypes.byref(s), None, None, None, None, None) == 1
    fake = ctypes.c_void_p(4096)       # never dereferenced: the call fails before any launch
    rc = r3.lib.r3_permute(ctypes.byref(s), fake, None, fake, fake, fake, fake, None, None, 0,
                           None, None)
    assert rc == 3                     # R3_ERR_WORKSPACE
    rc = r3.lib.r3_grouped_swiglu(ctypes.byref(s), fake, fake, fake, fake, fake, fake, fake, 8,
                                  None, None)
    assert rc == 3
    big = r3.make_shape(16, 64, 2000, 2, 64, idx=__import__("torch").int16)
    assert r3.lib.r3_permute(ctypes.byref(big), fake, None, fake, fake, fake, fake, None, fake,
                             1 << 20, None, None) == 2      # R3_ERR_UNSUPPORTED
    with pytest.raises(ValueError):
        import torch
        r3.replay_gate_fwd(s, torch.zeros(16, 8), torch.zeros(16, 2, dtype=torch.uint8))


def test_workspace_sizes_scale_with_the_layer(r3):
    s = r3.make_shape(4096, 2048, 128, 8, 768)
    R = 4096 * 8
    assert r3.grouped_swiglu_workspace_bytes(s) >= R * 768 * 2
    assert r3.replay_layer_workspace_bytes(s) >= 2 * R * 2048 * 2 + R * 768 * 2
    assert r3.replay_layer_host_workspace_bytes(s) > r3.replay_layer_workspace_bytes(s)
    assert r3.permute_workspace_bytes(s) == 128 * 16 * 4


def test_host_call_chunk_schedule(r3):
    """r3_replay_layer_host_chunks: one chunk below 16384 tokens; above, chunks that cover
    [0, T) without gaps, start on multiples of 256, number at most 16, and end with small ones."""
    for T in (1, 300, 8192, 16383):
        assert r3.replay_layer_host_chunks(r3.make_shape(T, 64, 16, 2, 64)) == [0, T]
    for T in (16384, 16385, 40000, 65536, 100000, 1 << 20):
        st = r3.replay_layer_host_chunks(r3.make_shape(T, 64, 16, 2, 64))
        sizes = [b - a for a, b in zip(st, st[1:])]
        assert st[0] == 0 and st[-1] == T and all(n > 0 for n in sizes)
        assert 2 <= len(sizes) <= 16
        assert all(a % 256 == 0 for a in st[:-1])
        assert sizes[-1] <= max(sizes) // 2 + 256
    assert r3.replay_layer_host_chunks(r3.make_shape(65536, 64, 16, 2, 64)) == \
        [0, 8192, 16384, 24576, 32768, 40960, 49152, 57344, 61440, 63488, 65536]
