"""Thin ctypes binding over libr3_b200.so (the C ABI declared in include/r3.h).

Argument marshalling only: every step of the replayed layer runs in the CUDA library.  PyTorch
supplies device memory and the current stream.  There is no CPU fallback: importing this module
without a built library raises, and every call requires CUDA tensors.
"""
from __future__ import annotations

import ctypes
import os

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libr3_b200.so")
if not os.path.exists(_LIB_PATH):
    raise ImportError(
        f"{_LIB_PATH} is missing: build it with `python -m paper_2510_11370_b200.build` "
        "(needs nvcc; there is no CPU fallback)")
lib = ctypes.CDLL(_LIB_PATH)

R3_OK = 0
R3_ERR_INVALID_ARG, R3_ERR_UNSUPPORTED, R3_ERR_WORKSPACE, R3_ERR_CUDA = 1, 2, 3, 4
R3_ERR_SCRATCH_LIMIT = 5
R3_ERR_OUT_OF_PAGES = 6
R3_F32, R3_BF16 = 0, 1
R3_IDX_U8, R3_IDX_I16 = 1, 2
DEV_OK, DEV_BAD_INDEX, DEV_DUP_INDEX, DEV_TIMEOUT = 0, 1, 2, 3

EXPORTS = [
    "r3_status_string", "r3_capture_topk", "r3_capture_topk_batched",
    "r3_capture_topk_workspace_bytes", "r3_capture_topk_ws", "r3_replay_gate_fwd",
    "r3_replay_gate_bwd", "r3_permute_workspace_bytes", "r3_permute", "r3_permute_static",
    "r3_grouped_swiglu_workspace_bytes", "r3_grouped_swiglu", "r3_grouped_swiglu_gather",
    "r3_expert_up_swiglu",
    "r3_expert_down", "r3_combine",
    "r3_combine_residual", "r3_combine_bwd_gates", "r3_replay_finish",
    "r3_replay_layer_workspace_bytes",
    "r3_replay_layer", "r3_replay_blocks", "r3_replay_stack_workspace_bytes", "r3_replay_stack",
    "r3_replay_layer_host_workspace_bytes", "r3_replay_layer_host", "r3_replay_layer_host_enqueue",
    "r3_replay_layer_host_chunks",
    "r3_replay_layer_same_record",
    "r3_prob_discrepancy_workspace_bytes", "r3_prob_discrepancy", "r3_record_diff",
    "r3_sequence_diff", "r3_grouped_swiglu_bwd_workspace_bytes", "r3_grouped_swiglu_bwd_input",
    "r3_grouped_swiglu_bwd", "r3_grouped_swiglu_train", "r3_scale_rows", "r3_input_grad_finish",
    "r3_replay_layer_train_workspace_bytes", "r3_replay_layer_train",
    "r3_replay_stack_train_workspace_bytes", "r3_replay_stack_train",
    "r3_ep_regroup_map", "r3_ep_move_rows", "r3_ep_dest_table", "r3_ep_dispatch_rows",
    "r3_ep_slot_rows", "r3_replay_finish_rows",
    "r3_record_page_bytes", "r3_record_append", "r3_record_gather",
    "r3_pagepool_create", "r3_pagepool_destroy", "r3_pagepool_free_pages", "r3_pagepool_match",
    "r3_pagepool_alloc", "r3_pagepool_publish", "r3_pagepool_release",
    "r3_selftest_bounded_wait",
]


class Shape(ctypes.Structure):
    _fields_ = [("T", ctypes.c_int32), ("d", ctypes.c_int32), ("E", ctypes.c_int32),
                ("K", ctypes.c_int32), ("F", ctypes.c_int32), ("act_dtype", ctypes.c_int32),
                ("router_w_dtype", ctypes.c_int32), ("idx_type", ctypes.c_int32)]


_P = ctypes.c_void_p
_SP = ctypes.POINTER(Shape)
lib.r3_status_string.restype = ctypes.c_char_p
lib.r3_status_string.argtypes = [ctypes.c_int]
lib.r3_grouped_swiglu_bwd_input.argtypes = [_SP] + [_P] * 9 + [ctypes.c_size_t, _P, _P]
lib.r3_grouped_swiglu_train.argtypes = [_SP] + [_P] * 9 + [ctypes.c_size_t, _P, _P]
lib.r3_scale_rows.argtypes = [_SP] + [_P] * 5
lib.r3_input_grad_finish.argtypes = [_SP] + [_P] * 12
lib.r3_replay_layer_train.argtypes = [_SP] + [_P] * 15 + [ctypes.c_size_t, _P, _P]
lib.r3_replay_stack_train_workspace_bytes.restype = ctypes.c_size_t
lib.r3_replay_stack_train_workspace_bytes.argtypes = [_SP, ctypes.c_int32]
lib.r3_replay_stack_train.argtypes = [_SP, ctypes.c_int32] + [_P] * 15 + [ctypes.c_size_t, _P, _P]
lib.r3_ep_regroup_map.argtypes = [_P, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, _P, _P, _P, _P]
lib.r3_ep_dest_table.argtypes = [_P, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, _P, _P, _P]
lib.r3_ep_dispatch_rows.argtypes = [_SP, ctypes.c_int32, _P, _P, _P, _P, _P, _P, ctypes.c_int64,
                                    _P, _P]
lib.r3_ep_slot_rows.argtypes = [_SP, ctypes.c_int32, _P, _P, _P, _P, _P, ctypes.c_int64, _P, _P, _P]
lib.r3_replay_finish_rows.argtypes = [_SP] + [_P] * 10
lib.r3_ep_move_rows.argtypes = [_P, _P, _P, ctypes.c_int32, ctypes.c_size_t, ctypes.c_int32, _P]
lib.r3_grouped_swiglu_bwd.argtypes = [_SP] + [_P] * 13 + [ctypes.c_size_t, _P, _P]
for _n in ("r3_permute_workspace_bytes", "r3_grouped_swiglu_workspace_bytes",
           "r3_grouped_swiglu_bwd_workspace_bytes", "r3_replay_layer_train_workspace_bytes",
           "r3_replay_stack_workspace_bytes",
           "r3_replay_layer_workspace_bytes", "r3_replay_layer_host_workspace_bytes"):
    getattr(lib, _n).restype = ctypes.c_size_t
    getattr(lib, _n).argtypes = [_SP]
lib.r3_capture_topk.argtypes = [_SP, _P, _P, _P, _P, _P]
lib.r3_capture_topk_batched.argtypes = [_SP, ctypes.c_int32, _P, _P, _P, _P, _P]
lib.r3_capture_topk_workspace_bytes.restype = ctypes.c_size_t
lib.r3_capture_topk_workspace_bytes.argtypes = [_SP, ctypes.c_int32]
lib.r3_capture_topk_ws.argtypes = [_SP, ctypes.c_int32, _P, _P, _P, _P, _P, ctypes.c_size_t, _P]
lib.r3_replay_gate_fwd.argtypes = [_SP, _P, _P, _P, _P, _P]
lib.r3_replay_gate_bwd.argtypes = [_SP, _P, _P, _P, _P, _P]
lib.r3_permute.argtypes = [_SP, _P, _P, _P, _P, _P, _P, _P, _P, ctypes.c_size_t, _P, _P]
lib.r3_permute_static.argtypes = [_SP, _P, _P, _P, _P, _P, _P, _P, _P, _P]
lib.r3_grouped_swiglu.argtypes = [_SP, _P, _P, _P, _P, _P, _P, _P, ctypes.c_size_t, _P, _P]
lib.r3_grouped_swiglu_gather.argtypes = [_SP, _P, _P, _P, _P, _P, _P, _P, _P, ctypes.c_size_t, _P, _P]
lib.r3_expert_up_swiglu.argtypes = [_SP, _P, _P, _P, _P, _P, ctypes.c_size_t, _P, _P]
lib.r3_expert_down.argtypes = [_SP, _P, _P, _P, ctypes.c_size_t, _P, _P]
lib.r3_combine.argtypes = [_SP, _P, _P, _P, _P, _P]
lib.r3_combine_residual.argtypes = [_SP, _P, _P, _P, _P, _P, _P]
lib.r3_replay_blocks.argtypes = [_SP, ctypes.c_int32] + [_P] * 10 + [ctypes.c_size_t, _P, _P]
lib.r3_replay_stack.argtypes = [_SP, ctypes.c_int32] + [_P] * 10 + [ctypes.c_size_t, _P, _P]
lib.r3_combine_bwd_gates.argtypes = [_SP, _P, _P, _P, _P, _P]
lib.r3_replay_finish.argtypes = [_SP] + [_P] * 11
lib.r3_replay_layer.argtypes = [_SP] + [_P] * 11 + [ctypes.c_size_t, _P, _P]
lib.r3_replay_layer_same_record.argtypes = [_SP] + [_P] * 11 + [ctypes.c_size_t, _P, _P]
lib.r3_replay_layer_host.argtypes = [_SP] + [_P] * 10 + [ctypes.c_size_t, _P, _P]
lib.r3_replay_layer_host_enqueue.argtypes = [_SP] + [_P] * 10 + [ctypes.c_size_t, _P, _P]
lib.r3_prob_discrepancy_workspace_bytes.restype = ctypes.c_size_t
lib.r3_prob_discrepancy_workspace_bytes.argtypes = [ctypes.c_int64]
lib.r3_prob_discrepancy.argtypes = [_P, _P, ctypes.c_int64, _P, ctypes.c_int32, _P, _P, _P,
                                    ctypes.c_size_t, _P]
lib.r3_record_diff.argtypes = [_SP, ctypes.c_int32, _P, _P, _P, _P, _P, _P, _P]
lib.r3_sequence_diff.argtypes = [_P, _P, ctypes.c_int32, _P, _P]
_I32 = ctypes.c_int32
lib.r3_record_page_bytes.restype = ctypes.c_size_t
lib.r3_record_page_bytes.argtypes = [_SP, _I32, _I32]
lib.r3_record_append.argtypes = [_SP, _I32, _I32, _I32, _P, _P, _I32, _P, _P, _I32, _P, _I32, _P, _P]
lib.r3_record_gather.argtypes = [_SP, _I32, _I32, _I32, _P, _P, _I32, _P, _I32, _P, _I32, _P, _P]
lib.r3_pagepool_create.restype = ctypes.c_void_p
lib.r3_pagepool_create.argtypes = [_I32, _I32]
lib.r3_pagepool_destroy.restype = None
lib.r3_pagepool_destroy.argtypes = [_P]
lib.r3_pagepool_free_pages.argtypes = [_P]
lib.r3_pagepool_match.argtypes = [_P, _P, _I32, _P, _I32]
lib.r3_pagepool_alloc.argtypes = [_P, _I32, _P]
lib.r3_pagepool_publish.argtypes = [_P, _P, _I32, _P, _I32]
lib.r3_pagepool_release.argtypes = [_P, _P, _I32]
lib.r3_selftest_bounded_wait.argtypes = [ctypes.c_int64, _P, _P, _P]
lib.r3_replay_layer_host_chunks.argtypes = [_SP, _P]
_NOT_STATUS = ("r3_status_string", "r3_pagepool_create", "r3_pagepool_destroy",
               "r3_replay_layer_host_chunks")
for _n in EXPORTS:
    if _n not in _NOT_STATUS and not _n.endswith("_bytes"):
        getattr(lib, _n).restype = ctypes.c_int


class R3Error(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__(lib.r3_status_string(code).decode())


def _check(code: int) -> None:
    if code != R3_OK:
        raise R3Error(code)


_ACT = {torch.float32: R3_F32, torch.bfloat16: R3_BF16}
_IDX = {torch.uint8: R3_IDX_U8, torch.int16: R3_IDX_I16}


def make_shape(T, d, E, K, F, act=torch.bfloat16, router=torch.float32, idx=torch.uint8) -> Shape:
    return Shape(T, d, E, K, F, _ACT[act], _ACT[router], _IDX[idx])


def shape_of(w) -> Shape:
    """Shape of a synth.Workload."""
    return make_shape(w.T, w.d, w.E, w.K, w.F, w.act_dtype, w.router_dtype, w.idx_dtype)


def _act_dtype(s: Shape):
    return torch.bfloat16 if s.act_dtype == R3_BF16 else torch.float32


def _idx_dtype(s: Shape):
    return torch.uint8 if s.idx_type == R3_IDX_U8 else torch.int16


def _ptr(t, host: bool = False):
    if t is None:
        return None
    if not isinstance(t, torch.Tensor):
        raise TypeError("expected a torch.Tensor")
    if host:
        if t.is_cuda:
            raise ValueError("expected a host tensor")
    elif not t.is_cuda:
        raise ValueError("expected a CUDA tensor (there is no CPU path)")
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream)


def _dev(*ts):
    for t in ts:
        if isinstance(t, torch.Tensor):
            return t.device
    return torch.device("cuda")


def workspace(nbytes: int, device) -> torch.Tensor:
    """Device scratch of at least nbytes, 256-byte aligned (torch's allocator aligns to 512)."""
    return torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def new_status(device) -> torch.Tensor:
    return torch.zeros(1, dtype=torch.int32, device=device)


# ---------------------------------------------------------------------------------------------
def capture_topk(s: Shape, x, w_router, idx_out=None, logits_out=None, *, want_idx=True,
                 want_logits=False, stream=None):
    """Router logits + TopKMask.  Returns (idx [T,K] or None, logits [T,E] or None)."""
    dev = _dev(x)
    if idx_out is None and want_idx:
        idx_out = torch.empty((s.T, s.K), dtype=_idx_dtype(s), device=dev)
    if logits_out is None and want_logits:
        logits_out = torch.empty((s.T, s.E), dtype=torch.float32, device=dev)
    _check(lib.r3_capture_topk(ctypes.byref(s), _ptr(x), _ptr(w_router), _ptr(idx_out),
                               _ptr(logits_out), _stream(stream)))
    return idx_out, logits_out


def capture_topk_batched(s: Shape, L: int, x, w_router, idx_out=None, logits_out=None, *,
                         want_idx=True, want_logits=False, stream=None):
    """L layers at once: x [L,T,d], w_router [L,E,d] -> idx [L,T,K], logits [L,T,E]."""
    dev = _dev(x)
    if idx_out is None and want_idx:
        idx_out = torch.empty((L, s.T, s.K), dtype=_idx_dtype(s), device=dev)
    if logits_out is None and want_logits:
        logits_out = torch.empty((L, s.T, s.E), dtype=torch.float32, device=dev)
    _check(lib.r3_capture_topk_batched(ctypes.byref(s), L, _ptr(x), _ptr(w_router),
                                       _ptr(idx_out), _ptr(logits_out), _stream(stream)))
    return idx_out, logits_out


def capture_topk_workspace_bytes(s: Shape, L: int = 1) -> int:
    return lib.r3_capture_topk_workspace_bytes(ctypes.byref(s), L)


def capture_topk_ws(s: Shape, L: int, x, w_router, idx_out=None, logits_out=None, *, ws=None,
                    want_idx=True, want_logits=False, stream=None):
    """capture_topk with scratch, so that float32 router weights run on the tensor cores too."""
    dev = _dev(x)
    lead = (L,) if x.dim() == 3 else ()
    if idx_out is None and want_idx:
        idx_out = torch.empty(lead + (s.T, s.K), dtype=_idx_dtype(s), device=dev)
    if logits_out is None and want_logits:
        logits_out = torch.empty(lead + (s.T, s.E), dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(capture_topk_workspace_bytes(s, L), dev)
    _check(lib.r3_capture_topk_ws(ctypes.byref(s), L, _ptr(x), _ptr(w_router), _ptr(idx_out),
                                  _ptr(logits_out), _ptr(ws), ws.numel(), _stream(stream)))
    return idx_out, logits_out


def replay_gate_fwd(s: Shape, logits, idx, gates=None, dev_status=None, stream=None):
    if gates is None:
        gates = torch.empty((s.T, s.K), dtype=torch.float32, device=_dev(logits))
    _check(lib.r3_replay_gate_fwd(ctypes.byref(s), _ptr(logits), _ptr(idx), _ptr(gates),
                                  _ptr(dev_status), _stream(stream)))
    return gates


def replay_gate_bwd(s: Shape, gates, dgates, idx, dlogits=None, stream=None):
    if dlogits is None:
        dlogits = torch.empty((s.T, s.E), dtype=torch.float32, device=_dev(gates))
    _check(lib.r3_replay_gate_bwd(ctypes.byref(s), _ptr(gates), _ptr(dgates), _ptr(idx),
                                  _ptr(dlogits), _stream(stream)))
    return dlogits


def permute_workspace_bytes(s: Shape) -> int:
    return lib.r3_permute_workspace_bytes(ctypes.byref(s))


def permute(s: Shape, idx, x=None, *, out=None, ws=None, dev_status=None, stream=None):
    """Returns (counts, offsets, row_of_slot, slot_of_row, xp or None)."""
    dev = _dev(idx)
    R = s.T * s.K
    if out is None:
        counts = torch.empty(s.E, dtype=torch.int32, device=dev)
        offsets = torch.empty(s.E + 1, dtype=torch.int32, device=dev)
        ros = torch.empty((s.T, s.K), dtype=torch.int32, device=dev)
        sor = torch.empty(R, dtype=torch.int32, device=dev)
        xp = torch.empty((R, s.d), dtype=_act_dtype(s), device=dev) if x is not None else None
    else:
        counts, offsets, ros, sor, xp = out
    if ws is None:
        ws = workspace(permute_workspace_bytes(s), dev)
    _check(lib.r3_permute(ctypes.byref(s), _ptr(idx), _ptr(x), _ptr(counts), _ptr(offsets),
                          _ptr(ros), _ptr(sor), _ptr(xp), _ptr(ws), ws.numel(),
                          _ptr(dev_status), _stream(stream)))
    return counts, offsets, ros, sor, xp


def permute_static(s: Shape, idx, x, counts, offsets, row_of_slot, slot_of_row, xp, *,
                   dev_status=None, stream=None):
    """r3_permute with the scratch inside the library: for callers that cannot allocate device
    memory where they call from (their memory belongs to someone else's pool, or was budgeted
    ahead of time).  All outputs are passed in; nothing is allocated here either.  Raises
    R3Error(R3_ERR_SCRATCH_LIMIT) when E * ceil(T / 256) > 262144.  Do not overlap calls."""
    _check(lib.r3_permute_static(ctypes.byref(s), _ptr(idx), _ptr(x), _ptr(counts),
                                 _ptr(offsets), _ptr(row_of_slot), _ptr(slot_of_row), _ptr(xp),
                                 _ptr(dev_status), _stream(stream)))
    return counts, offsets, row_of_slot, slot_of_row, xp


def grouped_swiglu_workspace_bytes(s: Shape) -> int:
    return lib.r3_grouped_swiglu_workspace_bytes(ctypes.byref(s))


def grouped_swiglu(s: Shape, xp, offsets, w_gate, w_up, w_down, o=None, *, ws=None,
                   dev_status=None, stream=None):
    dev = _dev(xp)
    if o is None:
        o = torch.empty((s.T * s.K, s.d), dtype=_act_dtype(s), device=dev)
    if ws is None:
        ws = workspace(grouped_swiglu_workspace_bytes(s), dev)
    _check(lib.r3_grouped_swiglu(ctypes.byref(s), _ptr(xp), _ptr(offsets), _ptr(w_gate),
                                 _ptr(w_up), _ptr(w_down), _ptr(o), _ptr(ws), ws.numel(),
                                 _ptr(dev_status), _stream(stream)))
    return o


def grouped_swiglu_gather(s: Shape, x, slot_of_row, offsets, w_gate, w_up, w_down, o=None, *,
                          ws=None, dev_status=None, stream=None):
    """grouped_swiglu reading the token rows in place from x [T,d] through slot_of_row (bf16)."""
    dev = _dev(x)
    if o is None:
        o = torch.empty((s.T * s.K, s.d), dtype=_act_dtype(s), device=dev)
    if ws is None:
        ws = workspace(grouped_swiglu_workspace_bytes(s), dev)
    _check(lib.r3_grouped_swiglu_gather(ctypes.byref(s), _ptr(x), _ptr(slot_of_row), _ptr(offsets),
                                        _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(o), _ptr(ws),
                                        ws.numel(), _ptr(dev_status), _stream(stream)))
    return o


def expert_up_swiglu(s: Shape, xp, offsets, w_gate, w_up, ws, dev_status=None, stream=None):
    """First half of grouped_swiglu: tile list + h = silu(xp Wg^T) * (xp Wu^T) into `ws`."""
    _check(lib.r3_expert_up_swiglu(ctypes.byref(s), _ptr(xp), _ptr(offsets), _ptr(w_gate),
                                   _ptr(w_up), _ptr(ws), ws.numel(), _ptr(dev_status),
                                   _stream(stream)))


def expert_down(s: Shape, w_down, o, ws, dev_status=None, stream=None):
    """Second half of grouped_swiglu: o = h W_down^T with h taken from `ws`."""
    _check(lib.r3_expert_down(ctypes.byref(s), _ptr(w_down), _ptr(o), _ptr(ws), ws.numel(),
                              _ptr(dev_status), _stream(stream)))
    return o


def combine(s: Shape, o, row_of_slot, gates, y=None, stream=None):
    if y is None:
        y = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=_dev(o))
    _check(lib.r3_combine(ctypes.byref(s), _ptr(o), _ptr(row_of_slot), _ptr(gates), _ptr(y),
                          _stream(stream)))
    return y


def combine_residual(s: Shape, o, row_of_slot, gates, residual, y=None, stream=None):
    """y = residual + sum_j gates[:, j] * o[row_of_slot[:, j]]."""
    if y is None:
        y = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=_dev(o))
    _check(lib.r3_combine_residual(ctypes.byref(s), _ptr(o), _ptr(row_of_slot), _ptr(gates),
                                   _ptr(residual), _ptr(y), _stream(stream)))
    return y


def replay_blocks(s: Shape, L: int, x, w_router, idx, w_gate, w_up, w_down, dy, *, y=None,
                  dlogits=None, ws=None, dev_status=None, stream=None):
    """L independent replayed blocks, all tensors stacked on a leading layer axis.
    Returns (y [L,T,d], dlogits [L,T,E])."""
    dev = _dev(x)
    if y is None:
        y = torch.empty((L, s.T, s.d), dtype=_act_dtype(s), device=dev)
    if dlogits is None:
        dlogits = torch.empty((L, s.T, s.E), dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(replay_layer_workspace_bytes(s), dev)
    _check(lib.r3_replay_blocks(ctypes.byref(s), L, _ptr(x), _ptr(w_router), _ptr(idx),
                                _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(dy), _ptr(y),
                                _ptr(dlogits), _ptr(ws), ws.numel(), _ptr(dev_status),
                                _stream(stream)))
    return y, dlogits


def replay_stack_workspace_bytes(s: Shape) -> int:
    return lib.r3_replay_stack_workspace_bytes(ctypes.byref(s))


def replay_stack(s: Shape, L: int, x0, w_router, idx, w_gate, w_up, w_down, dy, *, x_out=None,
                 dlogits=None, ws=None, dev_status=None, stream=None):
    """L residual MoE blocks with replayed routing.  Returns (x_L [T,d], dlogits [L,T,E])."""
    dev = _dev(x0)
    if x_out is None:
        x_out = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    if dlogits is None:
        dlogits = torch.empty((L, s.T, s.E), dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(replay_stack_workspace_bytes(s), dev)
    _check(lib.r3_replay_stack(ctypes.byref(s), L, _ptr(x0), _ptr(w_router), _ptr(idx),
                               _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(dy), _ptr(x_out),
                               _ptr(dlogits), _ptr(ws), ws.numel(), _ptr(dev_status),
                               _stream(stream)))
    return x_out, dlogits


def combine_bwd_gates(s: Shape, dy, o, row_of_slot, dgates=None, stream=None):
    if dgates is None:
        dgates = torch.empty((s.T, s.K), dtype=torch.float32, device=_dev(o))
    _check(lib.r3_combine_bwd_gates(ctypes.byref(s), _ptr(dy), _ptr(o), _ptr(row_of_slot),
                                    _ptr(dgates), _stream(stream)))
    return dgates


def replay_finish(s: Shape, logits, idx, o, row_of_slot, dy, *, residual=None, y=None, gates=None,
                  dlogits=None, dev_status=None, stream=None):
    """Replay gate + combine + gate gradient + router-logit gradient in one pass over `o`
    (K <= 8).  Returns (y, gates, dlogits)."""
    dev = _dev(o)
    if y is None:
        y = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    if gates is None:
        gates = torch.empty((s.T, s.K), dtype=torch.float32, device=dev)
    if dlogits is None:
        dlogits = torch.empty((s.T, s.E), dtype=torch.float32, device=dev)
    _check(lib.r3_replay_finish(ctypes.byref(s), _ptr(logits), _ptr(idx), _ptr(o),
                                _ptr(row_of_slot), _ptr(dy), _ptr(residual), _ptr(y), _ptr(gates),
                                _ptr(dlogits), _ptr(dev_status), _stream(stream)))
    return y, gates, dlogits


def replay_layer_workspace_bytes(s: Shape) -> int:
    return lib.r3_replay_layer_workspace_bytes(ctypes.byref(s))


def replay_layer(s: Shape, x, w_router, idx, w_gate, w_up, w_down, dy, *, y=None, dlogits=None,
                 gates=None, ws=None, dev_status=None, stream=None):
    """Forward + router-logit backward of the replayed layer.  Returns (y, dlogits, gates)."""
    dev = _dev(x)
    if y is None:
        y = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    if dlogits is None:
        dlogits = torch.empty((s.T, s.E), dtype=torch.float32, device=dev)
    if gates is None:
        gates = torch.empty((s.T, s.K), dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(replay_layer_workspace_bytes(s), dev)
    _check(lib.r3_replay_layer(ctypes.byref(s), _ptr(x), _ptr(w_router), _ptr(idx), _ptr(w_gate),
                               _ptr(w_up), _ptr(w_down), _ptr(dy), _ptr(y), _ptr(dlogits),
                               _ptr(gates), _ptr(ws), ws.numel(), _ptr(dev_status),
                               _stream(stream)))
    return y, dlogits, gates


def replay_layer_same_record(s: Shape, x, w_router, idx, w_gate, w_up, w_down, dy, *, ws, y=None,
                             dlogits=None, gates=None, dev_status=None, stream=None):
    """replay_layer for another pass over the record of the preceding replay_layer call on `ws`:
    the dispatch and the expert work lists left there are used again."""
    dev = _dev(x)
    if y is None:
        y = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    if dlogits is None:
        dlogits = torch.empty((s.T, s.E), dtype=torch.float32, device=dev)
    if gates is None:
        gates = torch.empty((s.T, s.K), dtype=torch.float32, device=dev)
    _check(lib.r3_replay_layer_same_record(ctypes.byref(s), _ptr(x), _ptr(w_router), _ptr(idx),
                                           _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(dy),
                                           _ptr(y), _ptr(dlogits), _ptr(gates), _ptr(ws),
                                           ws.numel(), _ptr(dev_status), _stream(stream)))
    return y, dlogits, gates


def replay_layer_host_workspace_bytes(s: Shape) -> int:
    return lib.r3_replay_layer_host_workspace_bytes(ctypes.byref(s))


def replay_layer_host_chunks(s: Shape) -> list:
    """Token offsets [0, ..., T] of the chunks r3_replay_layer_host sends one after the other."""
    starts = (ctypes.c_int64 * 17)()
    lib.r3_replay_layer_host_chunks.restype = ctypes.c_int32
    n = lib.r3_replay_layer_host_chunks(ctypes.byref(s), starts)
    if n <= 0:
        raise R3Error(1)
    return [int(starts[i]) for i in range(n + 1)]


def replay_layer_host(s: Shape, x_host, w_router, idx_host, w_gate, w_up, w_down, dy_host,
                      y_host, dlogits_host, *, ws, dev_status=None, stream=None):
    """As replay_layer with x, idx, dy, y, dlogits in (pinned) host memory; synchronises."""
    _check(lib.r3_replay_layer_host(ctypes.byref(s), _ptr(x_host, True), _ptr(w_router),
                                    _ptr(idx_host, True), _ptr(w_gate), _ptr(w_up), _ptr(w_down),
                                    _ptr(dy_host, True), _ptr(y_host, True),
                                    _ptr(dlogits_host, True), _ptr(ws), ws.numel(),
                                    _ptr(dev_status), _stream(stream)))
    return y_host, dlogits_host


def replay_layer_host_enqueue(s: Shape, x_host, w_router, idx_host, w_gate, w_up, w_down, dy_host,
                              y_host, dlogits_host, *, ws, dev_status=None, stream=None):
    """As replay_layer_host without the final synchronisation: the result is in y_host and
    dlogits_host once `stream` has been synchronised."""
    _check(lib.r3_replay_layer_host_enqueue(ctypes.byref(s), _ptr(x_host, True), _ptr(w_router),
                                            _ptr(idx_host, True), _ptr(w_gate), _ptr(w_up),
                                            _ptr(w_down), _ptr(dy_host, True), _ptr(y_host, True),
                                            _ptr(dlogits_host, True), _ptr(ws), ws.numel(),
                                            _ptr(dev_status), _stream(stream)))
    return y_host, dlogits_host


# ---------------------------------------------------------------------------------------------
def prob_discrepancy(p_train, p_infer, taus, *, kl=None, counts=None, ws=None, stream=None):
    """k3 KL estimate (Eq. kl) and extreme-token counts (Eq. etdf) of two float32 probability
    arrays.  `taus`: a list or a float32 device tensor.  Returns (kl [1] float64, counts [n_tau]
    int64); F(tau) = counts / n."""
    dev = _dev(p_train)
    n = p_train.numel()
    if not (isinstance(taus, torch.Tensor) and taus.is_cuda and taus.dtype == torch.float32):
        taus = torch.as_tensor(taus, dtype=torch.float32, device=dev).contiguous()
    if kl is None:
        kl = torch.empty(1, dtype=torch.float64, device=dev)
    if counts is None:
        counts = torch.empty(taus.numel(), dtype=torch.int64, device=dev)
    if ws is None:
        ws = workspace(lib.r3_prob_discrepancy_workspace_bytes(n), dev)
    _check(lib.r3_prob_discrepancy(_ptr(p_train), _ptr(p_infer), n, _ptr(taus), taus.numel(),
                                   _ptr(kl), _ptr(counts), _ptr(ws), ws.numel(), _stream(stream)))
    return kl, counts


def record_diff(s: Shape, L: int, rec_a, rec_b, *, want_diff=True, stream=None):
    """Differing expert choices between two records [L,T,K].  Returns (diff [L,T] uint8 or None,
    token_choices [T], token_routers [T], hist [K+1] int64)."""
    dev = _dev(rec_a)
    diff = torch.empty((L, s.T), dtype=torch.uint8, device=dev) if want_diff else None
    choices = torch.empty(s.T, dtype=torch.int32, device=dev)
    routers = torch.empty(s.T, dtype=torch.int32, device=dev)
    hist = torch.empty(s.K + 1, dtype=torch.int64, device=dev)
    _check(lib.r3_record_diff(ctypes.byref(s), L, _ptr(rec_a), _ptr(rec_b), _ptr(diff),
                              _ptr(choices), _ptr(routers), _ptr(hist), _stream(stream)))
    return diff, choices, routers, hist


def sequence_diff(token_routers, cu_seqlens, *, stream=None):
    """Per-sequence sums of token_routers over [cu_seqlens[s], cu_seqlens[s+1])."""
    S = cu_seqlens.numel() - 1
    out = torch.empty(S, dtype=torch.int64, device=_dev(token_routers))
    _check(lib.r3_sequence_diff(_ptr(token_routers), _ptr(cu_seqlens), S, _ptr(out),
                                _stream(stream)))
    return out


# ---------------------------------------------------------------------------------------------
def record_page_bytes(s: Shape, L: int, page_tokens: int) -> int:
    return lib.r3_record_page_bytes(ctypes.byref(s), L, page_tokens)


def record_append(s: Shape, L: int, page_tokens: int, pages, block_table, seq_pos0, cu_new,
                  rec_new, *, dev_status=None, stream=None):
    """Writes rec_new [L, N, K] (N new tokens, packed by cu_new) into the pages of their sequences."""
    n_pages = pages.numel() // record_page_bytes(s, L, page_tokens)
    B, max_pages = block_table.shape
    _check(lib.r3_record_append(ctypes.byref(s), L, page_tokens, n_pages, _ptr(pages),
                                _ptr(block_table), max_pages, _ptr(seq_pos0), _ptr(cu_new), B,
                                _ptr(rec_new), rec_new.shape[1], _ptr(dev_status), _stream(stream)))


def record_gather(s: Shape, L: int, page_tokens: int, pages, block_table, cu_seqlens, T: int, *,
                  out=None, dev_status=None, stream=None):
    """The packed record [L, T, K] of a variable-length batch, assembled from the pages."""
    n_pages = pages.numel() // record_page_bytes(s, L, page_tokens)
    B, max_pages = block_table.shape
    if out is None:
        out = torch.empty((L, T, s.K), dtype=_idx_dtype(s), device=_dev(pages))
    _check(lib.r3_record_gather(ctypes.byref(s), L, page_tokens, n_pages, _ptr(pages),
                                _ptr(block_table), max_pages, _ptr(cu_seqlens), B, _ptr(out), T,
                                _ptr(dev_status), _stream(stream)))
    return out


class PagePool:
    """Host-side page bookkeeping of the record store (r3_pagepool_*): lists in, lists out."""

    def __init__(self, n_pages: int, page_tokens: int):
        self.page_tokens = page_tokens
        self._h = lib.r3_pagepool_create(n_pages, page_tokens)
        if not self._h:
            raise ValueError("r3_pagepool_create failed")

    def close(self):
        if self._h:
            lib.r3_pagepool_destroy(self._h)
            self._h = None

    __del__ = close

    @staticmethod
    def _arr(v):
        return (ctypes.c_int32 * max(len(v), 1))(*v)

    def free_pages(self) -> int:
        return lib.r3_pagepool_free_pages(self._h)

    def match(self, token_ids) -> list:
        cap = len(token_ids) // self.page_tokens
        out = (ctypes.c_int32 * max(cap, 1))()
        n = lib.r3_pagepool_match(self._h, self._arr(token_ids), len(token_ids), out, cap)
        return list(out[:n])

    def alloc(self, n: int) -> list:
        out = (ctypes.c_int32 * max(n, 1))()
        _check(lib.r3_pagepool_alloc(self._h, n, out))
        return list(out[:n])

    def publish(self, token_ids, table) -> None:
        _check(lib.r3_pagepool_publish(self._h, self._arr(token_ids), len(token_ids),
                                       self._arr(table), len(table)))

    def release(self, table) -> None:
        _check(lib.r3_pagepool_release(self._h, self._arr(table), len(table)))


def grouped_swiglu_train(s: Shape, xp, offsets, w_gate, w_up, w_down, *, ws=None, dev_status=None,
                         stream=None):
    """Grouped experts that also return the pre-activations: (o [R,d], pre_gate, pre_up [R,F])."""
    dev = _dev(xp)
    R = s.T * s.K
    o = torch.empty((R, s.d), dtype=_act_dtype(s), device=dev)
    pre_gate = torch.empty((R, s.F), dtype=_act_dtype(s), device=dev)
    pre_up = torch.empty((R, s.F), dtype=_act_dtype(s), device=dev)
    if ws is None:
        ws = workspace(lib.r3_grouped_swiglu_workspace_bytes(ctypes.byref(s)), dev)
    _check(lib.r3_grouped_swiglu_train(ctypes.byref(s), _ptr(xp), _ptr(offsets), _ptr(w_gate),
                                       _ptr(w_up), _ptr(w_down), _ptr(o), _ptr(pre_gate),
                                       _ptr(pre_up), _ptr(ws), ws.numel(), _ptr(dev_status),
                                       _stream(stream)))
    return o, pre_gate, pre_up


def scale_rows(s: Shape, dy, gates, row_of_slot, dout=None, *, stream=None):
    """dout[row_of_slot[t,j]] = gates[t,j] * dy[t]."""
    if dout is None:
        dout = torch.empty((s.T * s.K, s.d), dtype=_act_dtype(s), device=_dev(dy))
    _check(lib.r3_scale_rows(ctypes.byref(s), _ptr(dy), _ptr(gates), _ptr(row_of_slot),
                             _ptr(dout), _stream(stream)))
    return dout


def input_grad_finish(s: Shape, dxp, row_of_slot, slot_of_row, offsets, dlogits, idx, x, w_router,
                      *, dx_residual=None, stream=None):
    """(dx [T,d], dw_router [E,d] float32) from the expert input gradient and dlogits."""
    dev = _dev(dxp)
    dx = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    dw_r = torch.empty((s.E, s.d), dtype=torch.float32, device=dev)
    _check(lib.r3_input_grad_finish(ctypes.byref(s), _ptr(dxp), _ptr(row_of_slot),
                                    _ptr(slot_of_row), _ptr(offsets), _ptr(dlogits), _ptr(idx),
                                    _ptr(x), _ptr(w_router), _ptr(dx_residual), _ptr(dx),
                                    _ptr(dw_r), _stream(stream)))
    return dx, dw_r


def grouped_swiglu_bwd(s: Shape, xp, dout, pre_gate, pre_up, offsets, w_gate, w_up, w_down, *,
                       ws=None, dev_status=None, stream=None):
    """Backward of the grouped experts: (dxp [R,d], dw_gate, dw_up [E,F,d], dw_down [E,d,F])."""
    dev = _dev(dout)
    dxp = torch.empty((s.T * s.K, s.d), dtype=_act_dtype(s), device=dev)
    dw_gate = torch.empty((s.E, s.F, s.d), dtype=torch.float32, device=dev)
    dw_up = torch.empty((s.E, s.F, s.d), dtype=torch.float32, device=dev)
    dw_down = torch.empty((s.E, s.d, s.F), dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(lib.r3_grouped_swiglu_bwd_workspace_bytes(ctypes.byref(s)), dev)
    _check(lib.r3_grouped_swiglu_bwd(ctypes.byref(s), _ptr(xp), _ptr(dout), _ptr(pre_gate),
                                     _ptr(pre_up), _ptr(offsets), _ptr(w_gate), _ptr(w_up),
                                     _ptr(w_down), _ptr(dxp), _ptr(dw_gate), _ptr(dw_up),
                                     _ptr(dw_down), _ptr(ws), ws.numel(), _ptr(dev_status),
                                     _stream(stream)))
    return dxp, dw_gate, dw_up, dw_down


def replay_layer_train(s: Shape, x, w_router, idx, w_gate, w_up, w_down, dy, *, ws=None,
                       dev_status=None, stream=None, expert_grads=False, dw_experts=None):
    """Forward and backward of one replayed layer: (y, dlogits, dx, dw_router), and with
    expert_grads also (dw_gate, dw_up, dw_down) appended (float32; `dw_experts` may supply the
    three output tensors)."""
    dev = _dev(x)
    y = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    dlogits = torch.empty((s.T, s.E), dtype=torch.float32, device=dev)
    dx = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    dw_r = torch.empty((s.E, s.d), dtype=torch.float32, device=dev)
    if ws is None:
        ws = workspace(lib.r3_replay_layer_train_workspace_bytes(ctypes.byref(s)), dev)
    dws = (None, None, None)
    if expert_grads:
        dws = dw_experts or (
            torch.empty((s.E, s.F, s.d), dtype=torch.float32, device=dev),
            torch.empty((s.E, s.F, s.d), dtype=torch.float32, device=dev),
            torch.empty((s.E, s.d, s.F), dtype=torch.float32, device=dev))
    _check(lib.r3_replay_layer_train(ctypes.byref(s), _ptr(x), _ptr(w_router), _ptr(idx),
                                     _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(dy), _ptr(y),
                                     _ptr(dlogits), _ptr(dx), _ptr(dw_r), _ptr(dws[0]),
                                     _ptr(dws[1]), _ptr(dws[2]), _ptr(ws), ws.numel(),
                                     _ptr(dev_status), _stream(stream)))
    if expert_grads:
        return (y, dlogits, dx, dw_r) + tuple(dws)
    return y, dlogits, dx, dw_r


def replay_stack_train(s: Shape, L, x0, w_router, idx, w_gate, w_up, w_down, dy, *, ws=None,
                       dev_status=None, stream=None, expert_grads=False):
    """L residual blocks forward, then the exact backward chain:
    (x_out, dlogits [L,T,E], dx0, dw_router [L,E,d]) (+ dw_gate, dw_up, dw_down)."""
    dev = _dev(x0)
    x_out = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    dx0 = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    dlogits = torch.empty((L, s.T, s.E), dtype=torch.float32, device=dev)
    dw_r = torch.empty((L, s.E, s.d), dtype=torch.float32, device=dev)
    dws = (None, None, None)
    if expert_grads:
        dws = (torch.empty((L, s.E, s.F, s.d), dtype=torch.float32, device=dev),
               torch.empty((L, s.E, s.F, s.d), dtype=torch.float32, device=dev),
               torch.empty((L, s.E, s.d, s.F), dtype=torch.float32, device=dev))
    if ws is None:
        ws = workspace(lib.r3_replay_stack_train_workspace_bytes(ctypes.byref(s), L), dev)
    _check(lib.r3_replay_stack_train(ctypes.byref(s), L, _ptr(x0), _ptr(w_router), _ptr(idx),
                                     _ptr(w_gate), _ptr(w_up), _ptr(w_down), _ptr(dy),
                                     _ptr(x_out), _ptr(dlogits), _ptr(dx0), _ptr(dw_r),
                                     _ptr(dws[0]), _ptr(dws[1]), _ptr(dws[2]), _ptr(ws),
                                     ws.numel(), _ptr(dev_status), _stream(stream)))
    if expert_grads:
        return (x_out, dlogits, dx0, dw_r) + dws
    return x_out, dlogits, dx0, dw_r


def ep_regroup_map(recv_counts, rows: int, *, dev_status=None, stream=None):
    """recv_counts [n_src, e_local] int32 (device) -> (perm [rows] int32, offsets [e_local+1])."""
    n_src, e_local = recv_counts.shape
    dev = _dev(recv_counts)
    perm = torch.empty(max(rows, 1), dtype=torch.int32, device=dev)[:rows]
    offsets = torch.empty(e_local + 1, dtype=torch.int32, device=dev)
    _check(lib.r3_ep_regroup_map(_ptr(recv_counts), n_src, e_local, rows,
                                 _ptr(perm) if rows else None, _ptr(offsets), _ptr(dev_status),
                                 _stream(stream)))
    return perm, offsets


def _peer_array(addresses):
    return (ctypes.c_uint64 * len(addresses))(*[int(a) for a in addresses])


def ep_dest_table(counts_all, rank: int, *, stream=None):
    """counts_all [n_ranks, E] int32 (device) -> (dst_base [E], offsets_local [E/n_ranks + 1])."""
    n, E = counts_all.shape
    dev = _dev(counts_all)
    dst_base = torch.empty(E, dtype=torch.int32, device=dev)
    offsets_local = torch.empty(E // n + 1, dtype=torch.int32, device=dev)
    _check(lib.r3_ep_dest_table(_ptr(counts_all), n, E, rank, _ptr(dst_base), _ptr(offsets_local),
                                _stream(stream)))
    return dst_base, offsets_local


def ep_dispatch_rows(s: Shape, n_ranks: int, x, idx, row_of_slot, my_offsets, dst_base,
                     peer_addresses, capacity_rows: int, *, dev_status=None, stream=None):
    """x[t] straight into the owners' receive buffers (peer_addresses: their base addresses,
    capacity_rows rows each; a row beyond the capacity is dropped and flagged)."""
    arr = _peer_array(peer_addresses)
    _check(lib.r3_ep_dispatch_rows(ctypes.byref(s), n_ranks, _ptr(x), _ptr(idx), _ptr(row_of_slot),
                                   _ptr(my_offsets), _ptr(dst_base), arr, int(capacity_rows),
                                   _ptr(dev_status), _stream(stream)))


def ep_slot_rows(s: Shape, n_ranks: int, idx, row_of_slot, my_offsets, dst_base, peer_addresses,
                 capacity_rows: int, *, dev_status=None, stream=None):
    """[T, K] addresses of the pairs' expert-output rows in the owners' output buffers."""
    row_ptr = torch.empty((s.T, s.K), dtype=torch.int64, device=_dev(idx))
    arr = _peer_array(peer_addresses)
    _check(lib.r3_ep_slot_rows(ctypes.byref(s), n_ranks, _ptr(idx), _ptr(row_of_slot),
                               _ptr(my_offsets), _ptr(dst_base), arr, int(capacity_rows),
                               _ptr(row_ptr), _ptr(dev_status), _stream(stream)))
    return row_ptr


def replay_finish_rows(s: Shape, logits, idx, row_ptr, dy, *, residual=None, dev_status=None,
                       stream=None):
    """r3_replay_finish with the expert-output rows given by address.  (y, gates, dlogits)."""
    dev = _dev(idx)
    y = torch.empty((s.T, s.d), dtype=_act_dtype(s), device=dev)
    gates = torch.empty((s.T, s.K), dtype=torch.float32, device=dev)
    dlogits = torch.empty((s.T, s.E), dtype=torch.float32, device=dev)
    _check(lib.r3_replay_finish_rows(ctypes.byref(s), _ptr(logits), _ptr(idx), _ptr(row_ptr),
                                     _ptr(dy), _ptr(residual), _ptr(y), _ptr(gates), _ptr(dlogits),
                                     _ptr(dev_status), _stream(stream)))
    return y, gates, dlogits


def ep_move_rows(src, perm, *, inverse=False, stream=None):
    """Rows of `src` [rows, width] reordered by `perm` (see r3_ep_move_rows)."""
    dst = torch.empty_like(src)
    rows = src.shape[0]
    if rows:
        _check(lib.r3_ep_move_rows(_ptr(src), _ptr(dst), _ptr(perm), rows,
                                   src.shape[1] * src.element_size(), 1 if inverse else 0,
                                   _stream(stream)))
    return dst


def grouped_swiglu_bwd_input(s: Shape, dout, pre_gate, pre_up, offsets, w_gate, w_up, w_down,
                             dxp=None, *, ws=None, dev_status=None, stream=None):
    """Input gradient of the grouped SwiGLU experts: dout [R,d] -> dxp [R,d] (bf16)."""
    dev = _dev(dout)
    if dxp is None:
        dxp = torch.empty((s.T * s.K, s.d), dtype=_act_dtype(s), device=dev)
    if ws is None:
        ws = workspace(lib.r3_grouped_swiglu_bwd_workspace_bytes(ctypes.byref(s)), dev)
    _check(lib.r3_grouped_swiglu_bwd_input(ctypes.byref(s), _ptr(dout), _ptr(pre_gate),
                                           _ptr(pre_up), _ptr(offsets), _ptr(w_gate), _ptr(w_up),
                                           _ptr(w_down), _ptr(dxp), _ptr(ws), ws.numel(),
                                           _ptr(dev_status), _stream(stream)))
    return dxp


def selftest_bounded_wait(limit_clocks: int, *, dev_status=None, device="cuda", stream=None):
    """Makes the library's bounded barrier wait run out on purpose (a barrier nothing signals).
    Returns out [4] int32: (wait result, abort flag, clocks waited, result of a second wait)."""
    out = torch.full((4,), -1, dtype=torch.int32, device=device)
    _check(lib.r3_selftest_bounded_wait(int(limit_clocks), _ptr(dev_status), _ptr(out),
                                        _stream(stream)))
    return out
