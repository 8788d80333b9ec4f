"""CPU oracle for the Rollout Routing Replay (R3) MoE layer.

TEST INFRASTRUCTURE ONLY.  This module is the slow, plain, float64 statement of what the
paper's Section 4.1 defines.  Only the test-suite, the smoke check and the benchmark's
``cpu_baseline`` / reference arm may import it; the product path (the CUDA library and its
Python binding) never does, and shares no code, table or constant with it.

Everything is numpy float64.  Inputs are the stored values of the tensors handed to the GPU
path (bf16 values widened exactly), so the only differences between the two sides are the
GPU's working precision and summation order.

Notation follows the paper: T tokens, hidden size d, M = E experts, K experts per token,
``s`` router logits, ``I`` the routing mask (kept as K indices per token), ``g`` gate weights,
``E_i`` the i-th expert network, ``y`` the layer output.  The expert network is a bias-free
SwiGLU feed-forward of width F (the paper leaves ``E_i`` abstract; the benchmark
configuration fixes it).

A library matmul / sort is used as a single step where the definition is a matrix product or
an ordering; there is no tiling, fusion or reordering beyond what the equations state.

Pins (see tests/test_oracle_pins.py): every public function is pinned to something other than
itself - closed forms, library routines on special cases, finite differences, brute force over
all M experts on tiny layers, and the stored golden values derived by hand in
tests/golden/.  No function here is "parity unpinned".
"""
from __future__ import annotations

import numpy as np

F64 = np.float64


def _f64(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=F64))


# ----------------------------------------------------------------------------------------------
# Section 4.1, first equation: router logits  s = x W_r
# ----------------------------------------------------------------------------------------------
def router_logits(x, w_r) -> np.ndarray:
    """s[t, i] = sum_c x[t, c] * W_r[i, c]   (Section 4.1, first equation).

    ``w_r`` is stored [E, d] (output-major), so the paper's ``x W_r`` is ``x @ w_r.T``.
    """
    return _f64(x) @ _f64(w_r).T


# ----------------------------------------------------------------------------------------------
# Section 4.1, second equation: I = TopKMask(s, K)
# ----------------------------------------------------------------------------------------------
def topk_indices(s, K: int) -> np.ndarray:
    """The K experts of TopKMask(s, K) for every token, as indices [T, K].

    Slot order is descending logit; exact ties go to the lower expert index (the paper does not
    state a tie rule; this is the reading used throughout).  A stable sort of the negated logits
    gives exactly that order.
    """
    s = _f64(s)
    T, E = s.shape
    if not 0 < K <= E:
        raise ValueError("need 0 < K <= E")
    order = np.argsort(-s, axis=1, kind="stable")
    return np.ascontiguousarray(order[:, :K]).astype(np.int64)


def mask_from_indices(idx, E: int) -> np.ndarray:
    """Binary mask I in {0,1}^M with exactly K ones per token (Section 4.1: sum_i I_i = K)."""
    idx = np.asarray(idx, dtype=np.int64)
    check_record(idx, E)
    T, K = idx.shape
    I = np.zeros((T, E), dtype=F64)
    I[np.arange(T)[:, None], idx] = 1.0
    return I


def check_record(idx, E: int) -> None:
    """A record is valid when every token lists K distinct experts in [0, E)."""
    idx = np.asarray(idx)
    if idx.ndim != 2:
        raise ValueError("record must be [T, K]")
    if idx.size and (idx.min() < 0 or idx.max() >= E):
        raise ValueError("expert index out of range")
    srt = np.sort(idx, axis=1)
    if idx.shape[1] > 1 and np.any(srt[:, 1:] == srt[:, :-1]):
        raise ValueError("duplicate expert in a token's record")


# ----------------------------------------------------------------------------------------------
# Eq. (train_gate) / Eq. (replay_gate): softmax of the training logits over a mask
# ----------------------------------------------------------------------------------------------
def gate_dense(s, I) -> np.ndarray:
    """g_i = I_i exp(s_i) / sum_j I_j exp(s_j), all M entries (Eq. train_gate / replay_gate).

    Written exactly as printed, over the dense mask.  The row maximum over the masked entries is
    subtracted first; that cancels in the ratio.
    """
    s = _f64(s)
    I = _f64(I)
    m = np.max(np.where(I > 0, s, -np.inf), axis=1, keepdims=True)
    num = I * np.exp(np.where(I > 0, s - m, 0.0))
    return num / np.sum(num, axis=1, keepdims=True)


def replay_gate(s_train, idx_infer) -> np.ndarray:
    """Eq. (replay_gate) restricted to the K recorded experts: gates [T, K], slot-aligned.

    g[t, j] = exp(s[t, e_j] - m) / sum_j' exp(s[t, e_j'] - m),  e_j = idx[t, j],
    m = max_j s[t, e_j].  The M - K other entries of the equation are zero and are not stored.
    """
    s = _f64(s_train)
    idx = np.asarray(idx_infer, dtype=np.int64)
    check_record(idx, s.shape[1])
    sel = np.take_along_axis(s, idx, axis=1)
    z = np.exp(sel - sel.max(axis=1, keepdims=True))
    return z / z.sum(axis=1, keepdims=True)


# ----------------------------------------------------------------------------------------------
# Expert network E_i (bias-free SwiGLU FFN, width F)
# ----------------------------------------------------------------------------------------------
def silu(z: np.ndarray) -> np.ndarray:
    return z / (1.0 + np.exp(-z))


def swiglu_expert(x, w_gate_i, w_up_i, w_down_i) -> np.ndarray:
    """E_i(x) = W_down,i ( silu(W_gate,i x) * (W_up,i x) ) for rows of x.

    w_gate_i, w_up_i: [F, d]; w_down_i: [d, F]  (all output-major).
    """
    x = _f64(x)
    a = x @ _f64(w_gate_i).T
    b = x @ _f64(w_up_i).T
    return (silu(a) * b) @ _f64(w_down_i).T


# ----------------------------------------------------------------------------------------------
# Eq. (replay_output):  y = sum_i g_replay,i E_i(x_train)
# ----------------------------------------------------------------------------------------------
def expert_outputs(x, idx, w_gate, w_up, w_down) -> np.ndarray:
    """E_{e_j}(x[t]) for every recorded (token, slot): array [T, K, d].

    These are the only terms of Eq. (replay_output) whose gate is non-zero.  The loop runs over
    experts i = 1..M as the sum in the equation does, evaluating expert i on the tokens whose
    mask has I_i = 1.
    """
    x = _f64(x)
    idx = np.asarray(idx, dtype=np.int64)
    T, K = idx.shape
    E = len(w_gate)
    check_record(idx, E)
    d_out = np.asarray(w_down[0]).shape[0]
    out = np.zeros((T, K, d_out), dtype=F64)
    for i in range(E):
        tt, jj = np.nonzero(idx == i)
        if tt.size == 0:
            continue
        out[tt, jj] = swiglu_expert(x[tt], w_gate[i], w_up[i], w_down[i])
    return out


def replay_output(x, s_train, idx_infer, w_gate, w_up, w_down):
    """Eq. (replay_output): y[t] = sum_j g[t, j] * E_{e_j}(x[t]).  Returns (y, gates, eo).

    ``eo`` is the [T, K, d] array of expert outputs, returned because the gradient needs it.
    """
    g = replay_gate(s_train, idx_infer)
    eo = expert_outputs(x, idx_infer, w_gate, w_up, w_down)
    y = np.einsum("tk,tkd->td", g, eo)
    return y, g, eo


def replay_output_dense(x, s_train, I_infer, w_gate, w_up, w_down) -> np.ndarray:
    """Eq. (replay_output) literally: sum over ALL M experts of g_replay,i E_i(x), dense mask.

    Every expert is evaluated on every token.  Tiny layers only.
    """
    x = _f64(x)
    g = gate_dense(s_train, I_infer)
    E = g.shape[1]
    y = np.zeros((x.shape[0], np.asarray(w_down[0]).shape[0]), dtype=F64)
    for i in range(E):
        y += g[:, i:i + 1] * swiglu_expert(x, w_gate[i], w_up[i], w_down[i])
    return y


def train_output(x, w_r, K, w_gate, w_up, w_down) -> np.ndarray:
    """The ordinary MoE layer, Eqs. (train_gate) and (train_output), written on its own:
    logits, TopKMask, softmax over the selected logits, weighted sum over all M experts."""
    s = router_logits(x, w_r)
    I = mask_from_indices(topk_indices(s, K), s.shape[1])
    return replay_output_dense(x, s, I, w_gate, w_up, w_down)


# ----------------------------------------------------------------------------------------------
# Token dispatch: the (expert, token) ordering implied by evaluating E_i only where I_i = 1
# ----------------------------------------------------------------------------------------------
def permutation(idx, E: int):
    """Stable grouping of the R = T*K (token, slot) pairs by expert.

    Pairs are listed in (t, j) order and stably sorted by key idx[t, j].  Returns
    counts [E], offsets [E+1] (exclusive scan), row_of_slot [T, K] (destination row of each
    pair) and slot_of_row [R] (flat pair index t*K + j held by each row), all int32.
    """
    idx = np.asarray(idx, dtype=np.int64)
    check_record(idx, E)
    T, K = idx.shape
    flat = idx.reshape(-1)
    slot_of_row = np.argsort(flat, kind="stable")
    row_of_slot = np.empty(T * K, dtype=np.int64)
    row_of_slot[slot_of_row] = np.arange(T * K)
    counts = np.bincount(flat, minlength=E)
    offsets = np.concatenate([[0], np.cumsum(counts)])
    return (counts.astype(np.int32), offsets.astype(np.int32),
            row_of_slot.reshape(T, K).astype(np.int32), slot_of_row.astype(np.int32))


def permute_rows(x, slot_of_row, K: int) -> np.ndarray:
    """xp[r] = x[token of row r]: the rows each expert reads, grouped by expert."""
    return np.asarray(x)[np.asarray(slot_of_row, dtype=np.int64) // K]


# ----------------------------------------------------------------------------------------------
# Router-logit gradient through the replayed mask (Section 4.1, purpose (b))
# ----------------------------------------------------------------------------------------------
def dgates(dy, eo) -> np.ndarray:
    """dL/dg[t, j] = <dy[t], E_{e_j}(x[t])>   (chain rule on Eq. replay_output)."""
    return np.einsum("td,tkd->tk", _f64(dy), _f64(eo))


def replay_gate_bwd(g, dg, idx, E: int) -> np.ndarray:
    """dL/ds_train [T, E] through Eq. (replay_gate) with I_infer held constant.

    On the mask d g_j / d s_{e_j'} = g_j (delta_jj' - g_j'), hence
    ds[t, e_j] = g_j (dg_j - sum_j' g_j' dg_j');  entries off the mask are zero.
    """
    g = _f64(g)
    dg = _f64(dg)
    idx = np.asarray(idx, dtype=np.int64)
    check_record(idx, E)
    T, K = idx.shape
    c = np.sum(g * dg, axis=1, keepdims=True)
    ds = np.zeros((T, E), dtype=F64)
    ds[np.arange(T)[:, None], idx] = g * (dg - c)
    return ds


def layer_fwd_bwd(x, w_r, idx_infer, w_gate, w_up, w_down, dy):
    """Whole replayed layer: forward (logits, gate, experts, output) and router-logit backward.

    Returns a dict with s, g, eo, y, dg, ds.
    """
    s = router_logits(x, w_r)
    y, g, eo = replay_output(x, s, idx_infer, w_gate, w_up, w_down)
    dg = dgates(dy, eo)
    ds = replay_gate_bwd(g, dg, idx_infer, s.shape[1])
    return dict(s=s, g=g, eo=eo, y=y, dg=dg, ds=ds)


def layer_tokens(x_rows, w_r, idx_rows, w_gate, w_up, w_down, dy_rows):
    """The same layer evaluated one token at a time, for spot checks at sizes where the whole
    batch is too slow: for each given token, K expert evaluations straight from the equations.
    Returns (y [n, d], ds [n, E])."""
    x_rows = _f64(x_rows)
    dy_rows = _f64(dy_rows)
    idx_rows = np.asarray(idx_rows, dtype=np.int64)
    n, K = idx_rows.shape
    E = len(w_gate)
    ys, dss = [], []
    for t in range(n):
        xt = x_rows[t:t + 1]
        s = router_logits(xt, w_r)
        g = replay_gate(s, idx_rows[t:t + 1])
        eo = np.stack([swiglu_expert(xt, w_gate[e], w_up[e], w_down[e])[0]
                       for e in idx_rows[t]])[None]
        ys.append(np.einsum("tk,tkd->td", g, eo)[0])
        dg = dgates(dy_rows[t:t + 1], eo)
        dss.append(replay_gate_bwd(g, dg, idx_rows[t:t + 1], E)[0])
    return np.stack(ys), np.stack(dss)


# ----------------------------------------------------------------------------------------------
# A stack of replayed MoE blocks with residual connections (benchmark configuration 5)
# ----------------------------------------------------------------------------------------------
def replay_stack_tokens(x_rows, layers, dy_rows, store=None):
    """Follows the given tokens through L residual blocks  x_{l+1} = store(x_l + y_replay,l(x_l)).

    Tokens are independent of each other in every step of the path, so a subset can be followed
    on its own.  ``layers`` is a sequence of (w_r, idx_rows, w_gate, w_up, w_down) per block, with
    idx_rows the record rows of these tokens.  ``dy_rows`` is the upstream gradient used for every
    block (the gradient arriving through the identity path).  ``store`` models the rounding of
    the stored activations (None = keep float64).  Returns (x_L rows, [ds_l rows for each l])."""
    x = _f64(x_rows)
    dss = []
    for (w_r, idx_rows, w_gate, w_up, w_down) in layers:
        y, ds = layer_tokens(x, w_r, idx_rows, w_gate, w_up, w_down, dy_rows)
        dss.append(ds)
        x = x + y
        if store is not None:
            x = _f64(store(x))
    return x, dss


# ----------------------------------------------------------------------------------------------
# Update-stage backward to the layer input and the router weight (Section 4.1, purpose (b):
# the mask I_infer is a constant, everything else is differentiated)
# ----------------------------------------------------------------------------------------------
def dsilu(z: np.ndarray) -> np.ndarray:
    """d silu / dz = sigma(z) (1 + z (1 - sigma(z)))."""
    sg = 1.0 / (1.0 + np.exp(-z))
    return sg * (1.0 + z * (1.0 - sg))


def swiglu_expert_bwd_input(x, do, w_gate_i, w_up_i, w_down_i) -> np.ndarray:
    """dL/dx for o = E_i(x) given dL/do, by the chain rule through
    a = W_gate x, b = W_up x, h = silu(a) b, o = W_down h."""
    x, do = _f64(x), _f64(do)
    wg, wu, wd = _f64(w_gate_i), _f64(w_up_i), _f64(w_down_i)
    a, b = x @ wg.T, x @ wu.T
    dh = do @ wd                                   # [n, F]
    da = dh * b * dsilu(a)
    db = dh * silu(a)
    return da @ wg + db @ wu


def layer_bwd_input(x, w_r, idx_infer, w_gate, w_up, w_down, dy):
    """Gradients of  L = <dy, y_replay(x)>  (any loss whose gradient at y is dy) with the recorded
    mask held constant:
        dx   [T, d]  = sum_j g_j dE_{e_j}/dx^T dy   (expert path)  +  ds W_r   (router path)
        dW_r [E, d]  = ds^T x
        ds   [T, E]  as replay_gate_bwd.
    Returns a dict with dx, dw_r, ds, dx_expert, dx_router."""
    x, dy, w_r = _f64(x), _f64(dy), _f64(w_r)
    idx = np.asarray(idx_infer, dtype=np.int64)
    T, K = idx.shape
    E = w_r.shape[0]
    f = layer_fwd_bwd(x, w_r, idx, w_gate, w_up, w_down, dy)
    dx_e = np.zeros_like(x)
    for i in range(E):
        tt, jj = np.nonzero(idx == i)
        if tt.size == 0:
            continue
        do = f["g"][tt, jj][:, None] * dy[tt]      # dL/d(E_i(x_t)) = g_{t,j} dy_t
        contrib = swiglu_expert_bwd_input(x[tt], do, w_gate[i], w_up[i], w_down[i])
        np.add.at(dx_e, tt, contrib)
    dx_r = f["ds"] @ w_r
    return dict(dx=dx_e + dx_r, dw_r=f["ds"].T @ x, ds=f["ds"], dx_expert=dx_e, dx_router=dx_r,
                y=f["y"], g=f["g"])


# ----------------------------------------------------------------------------------------------
# Update-stage backward to the expert weights (Section 4.1, purpose (b): with the mask replayed,
# the experts that receive a gradient are exactly those the rollout activated)
# ----------------------------------------------------------------------------------------------
def swiglu_expert_bwd_weights(x, do, w_gate_i, w_up_i, w_down_i):
    """(dW_gate_i [F,d], dW_up_i [F,d], dW_down_i [d,F]) for o = E_i(x) given dL/do over the n
    tokens routed to expert i:  a = W_gate x, b = W_up x, h = silu(a) b, o = W_down h, so
        dW_down = do^T h,  dh = do W_down,  da = dh b silu'(a),  db = dh silu(a),
        dW_gate = da^T x,  dW_up = db^T x."""
    x, do = _f64(x), _f64(do)
    wg, wu, wd = _f64(w_gate_i), _f64(w_up_i), _f64(w_down_i)
    a, b = x @ wg.T, x @ wu.T
    h = silu(a) * b
    dh = do @ wd
    da = dh * b * dsilu(a)
    db = dh * silu(a)
    return da.T @ x, db.T @ x, do.T @ h


def layer_bwd_weights(x, w_r, idx_infer, w_gate, w_up, w_down, dy, experts=None):
    """Expert-weight gradients of L = <dy, y_replay(x)> with the recorded mask held constant.
    Expert i sees the tokens whose record holds i, each with dL/do = g_{t,j} dy_t; an expert that
    no record names gets a zero gradient.  `experts` limits the work to those expert ids.
    Returns {i: (dW_gate_i, dW_up_i, dW_down_i)}."""
    x, dy, w_r = _f64(x), _f64(dy), _f64(w_r)
    idx = np.asarray(idx_infer, dtype=np.int64)
    E = w_r.shape[0]
    g = replay_gate(router_logits(x, w_r), idx)
    out = {}
    for i in (range(E) if experts is None else experts):
        tt, jj = np.nonzero(idx == i)
        do = g[tt, jj][:, None] * dy[tt]
        out[int(i)] = swiglu_expert_bwd_weights(x[tt], do, w_gate[i], w_up[i], w_down[i])
    return out


# ----------------------------------------------------------------------------------------------
# The exact backward chain of a stack of residual replayed blocks (benchmark configuration 5)
# ----------------------------------------------------------------------------------------------
def replay_stack_bwd_tokens(x_rows, layers, dy_rows, store=None, expert_grads=False):
    """x_{l+1} = store(x_l + y_replay,l(x_l)) for L blocks, then the gradient of
    <dy, x_L> back through every block with the recorded masks held constant:
        g_L = dy,   g_l = store(g_{l+1} + dx_l(g_{l+1}))
    where dx_l, ds_l, dW_r,l are layer_bwd_input of block l at its input x_l with upstream
    gradient g_{l+1} (the residual path carries g_{l+1} unchanged).  Tokens are independent, so a
    subset can be followed on its own; dW_r,l then holds the sum over these tokens only.
    With expert_grads, dw_experts[l] = layer_bwd_weights of block l at (x_l, g_{l+1}).
    Returns dict(x_out, dx0, ds=[...], dw_r=[...], dw_experts=[...]) with one entry per block."""
    x = _f64(x_rows)
    xs = []
    for (w_r, idx_rows, w_gate, w_up, w_down) in layers:
        xs.append(x)
        s = router_logits(x, w_r)
        y, _, _ = replay_output(x, s, np.asarray(idx_rows, dtype=np.int64), w_gate, w_up, w_down)
        x = x + y
        if store is not None:
            x = _f64(store(x))
    g = _f64(dy_rows)
    dss, dwrs, dwes = [None] * len(layers), [None] * len(layers), [None] * len(layers)
    for l in range(len(layers) - 1, -1, -1):
        w_r, idx_rows, w_gate, w_up, w_down = layers[l]
        res = layer_bwd_input(xs[l], w_r, idx_rows, w_gate, w_up, w_down, g)
        dss[l], dwrs[l] = res["ds"], res["dw_r"]
        if expert_grads:
            dwes[l] = layer_bwd_weights(xs[l], w_r, idx_rows, w_gate, w_up, w_down, g)
        g = g + res["dx"]
        if store is not None:
            g = _f64(store(g))
    return dict(x_out=x, dx0=g, ds=dss, dw_r=dwrs, dw_experts=dwes)
