"""Seeded synthetic inputs shaped like the paper's MoE workloads.

This module only draws random tensors and assembles routing records from logits that the
caller supplies.  It contains none of the replayed layer's arithmetic (no gate, no expert, no
gradient), so both the CUDA path and the CPU checker can be fed from it.

The paper evaluates on rollouts of a 128-expert / top-8 MoE language model; no dataset item,
prompt or trained weight is used here.  What is reproduced is the *shape* of the work
(tokens x hidden, expert count, top-k, FFN width) and the statistics of routing drift between
the inference and training engines (Section 3.2: about one router decision in ten differs),
emulated by adding Gaussian noise to the logits before the inference-side top-k.

Draw order and seeds: tensor ``name`` of layer ``l`` in a configuration with base seed ``s``
is drawn from ``torch.Generator(device).manual_seed(s * 1_000_003 + l * 101 + TENSOR_ID[name])``
with ``torch.randn`` in float32, scaled, then rounded to the storage dtype.
"""
from __future__ import annotations

from dataclasses import dataclass

import torch

TENSOR_ID = {"x": 1, "w_r": 2, "w_gate": 3, "w_up": 4, "w_down": 5, "dy": 6,
             "noise": 7, "perm": 8, "resample": 9}


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes follow the five configurations of the build brief)."""
    name: str
    T: int
    d: int
    E: int
    K: int
    F: int
    act: str = "bf16"          # storage dtype of x, expert weights, outputs: "bf16" | "f32"
    router_w: str = "f32"      # storage dtype of W_r
    record: str = "noise"      # "noise" | "resample"
    sigma: float = 0.05        # std of the logit noise that emulates inference-engine drift
    zipf_s: float = 0.0        # > 0: selection-only expert bias, popularity ~ Zipf(s)
    resample_frac: float = 0.1
    layers: int = 1
    seed: int = 0

    @property
    def idx_dtype(self) -> torch.dtype:
        return torch.uint8 if self.E <= 256 else torch.int16

    @property
    def act_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.act == "bf16" else torch.float32

    @property
    def router_dtype(self) -> torch.dtype:
        return torch.bfloat16 if self.router_w == "bf16" else torch.float32


WORKLOADS = {
    # config 1: tiny fp32 layer, record = own top-2 with 10% of tokens perturbed
    "c1_tiny_fp32": Workload("c1_tiny_fp32", T=512, d=128, E=8, K=2, F=256, act="f32",
                             record="resample"),
    # config 2: the headline single layer
    "c2_layer_bf16": Workload("c2_layer_bf16", T=4096, d=2048, E=128, K=8, F=768, sigma=0.05),
    # config 3: skewed routing
    "c3_skewed": Workload("c3_skewed", T=32768, d=2048, E=128, K=8, F=768, sigma=0.1,
                          zipf_s=1.2),
    # config 4: capture (decode batch, 48 layers, bf16 router) ...
    "c4_capture": Workload("c4_capture", T=256, d=2048, E=128, K=8, F=768, router_w="bf16",
                           layers=48),
    # ... and replay of a recorded 65536-token batch
    "c4_replay": Workload("c4_replay", T=65536, d=2048, E=128, K=8, F=768, router_w="bf16"),
    # config 5: 48 MoE blocks
    "c5_stack48": Workload("c5_stack48", T=16384, d=2048, E=128, K=8, F=768, layers=48),
}


def _gen(w: Workload, name: str, layer: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(w.seed * 1_000_003 + layer * 101 + TENSOR_ID[name])
    return g


def _randn(w: Workload, name: str, layer: int, shape, std: float, dtype, device) -> torch.Tensor:
    out = torch.empty(shape, dtype=dtype, device=device)
    g = _gen(w, name, layer, device)
    # draw in slabs so that multi-GB tensors never need a float32 copy of the whole thing
    flat = out.view(-1)
    slab = 1 << 26
    for lo in range(0, flat.numel(), slab):
        n = min(slab, flat.numel() - lo)
        flat[lo:lo + n] = (torch.randn(n, generator=g, device=device, dtype=torch.float32)
                           * std).to(dtype)
    return out


def activations(w: Workload, device="cpu", layer: int = 0) -> torch.Tensor:
    """x [T, d] ~ N(0, 1)."""
    return _randn(w, "x", layer, (w.T, w.d), 1.0, w.act_dtype, device)


def upstream_grad(w: Workload, device="cpu", layer: int = 0) -> torch.Tensor:
    """dy [T, d] ~ N(0, 1): the gradient arriving at the layer output."""
    return _randn(w, "dy", layer, (w.T, w.d), 1.0, w.act_dtype, device)


def router_weight(w: Workload, device="cpu", layer: int = 0) -> torch.Tensor:
    """W_r [E, d] ~ N(0, 0.02)."""
    return _randn(w, "w_r", layer, (w.E, w.d), 0.02, w.router_dtype, device)


def expert_weights(w: Workload, device="cpu", layer: int = 0):
    """(W_gate [E, F, d], W_up [E, F, d], W_down [E, d, F]) ~ N(0, 0.02)."""
    return (_randn(w, "w_gate", layer, (w.E, w.F, w.d), 0.02, w.act_dtype, device),
            _randn(w, "w_up", layer, (w.E, w.F, w.d), 0.02, w.act_dtype, device),
            _randn(w, "w_down", layer, (w.E, w.d, w.F), 0.02, w.act_dtype, device))


def drift_noise(w: Workload, device="cpu", layer: int = 0) -> torch.Tensor:
    """[T, E] float32 N(0, sigma^2), added to the logits before the inference-side top-k."""
    return _randn(w, "noise", layer, (w.T, w.E), w.sigma, torch.float32, device)


def zipf_bias(w: Workload, device="cpu", layer: int = 0) -> torch.Tensor:
    """Selection-only expert bias b_e = -s * ln(1 + pi(e)), pi a seeded permutation of 0..E-1.

    The bias enters only the synthetic inference-side selection (which experts get recorded);
    the layer itself stays bias-free as in the paper.  Zero when ``zipf_s == 0``.
    """
    if w.zipf_s <= 0:
        return torch.zeros(w.E, dtype=torch.float32, device=device)
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed * 1_000_003 + layer * 101 + TENSOR_ID["perm"])
    pi = torch.randperm(w.E, generator=g).to(torch.float32)
    return (-w.zipf_s * torch.log1p(pi)).to(device)


def select_top(scores: torch.Tensor, K: int, dtype: torch.dtype) -> torch.Tensor:
    """Indices of the K largest scores per row (descending, stable: ties to the lower index)."""
    order = torch.sort(scores, dim=1, descending=True, stable=True).indices
    return order[:, :K].contiguous().to(dtype)


def drifted_record(w: Workload, logits: torch.Tensor, layer: int = 0) -> torch.Tensor:
    """Record of an emulated inference engine: top-K of (given logits + bias + noise).

    ``logits`` [T, E] is supplied by the caller (float32 or float64, any device)."""
    dev = logits.device
    noise = drift_noise(w, dev, layer).to(logits.dtype)
    bias = zipf_bias(w, dev, layer).to(logits.dtype)
    return select_top(logits + bias[None, :] + noise, w.K, w.idx_dtype)


def resampled_record(w: Workload, own_topk: torch.Tensor, layer: int = 0) -> torch.Tensor:
    """Config-1 record: the given top-K, with a Bernoulli(resample_frac) subset of tokens having
    one uniformly chosen slot replaced by a uniform draw from the E-K experts not in their set."""
    g = torch.Generator(device="cpu")
    g.manual_seed(w.seed * 1_000_003 + layer * 101 + TENSOR_ID["resample"])
    idx = own_topk.to("cpu", torch.int64).clone()
    T, K = idx.shape
    hit = torch.rand(T, generator=g) < w.resample_frac
    slot = torch.randint(0, K, (T,), generator=g)
    pick = torch.randint(0, w.E - K, (T,), generator=g)
    for t in torch.nonzero(hit).flatten().tolist():
        others = [e for e in range(w.E) if e not in set(idx[t].tolist())]
        idx[t, slot[t]] = others[pick[t]]
    return idx.to(w.idx_dtype).to(own_topk.device)


def make_record(w: Workload, logits: torch.Tensor, layer: int = 0) -> torch.Tensor:
    """The replay record for a workload, built from logits supplied by the caller."""
    if w.record == "resample":
        own = select_top(logits, w.K, torch.int64)
        return resampled_record(w, own, layer)
    return drifted_record(w, logits, layer)


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (smaller T for quick cases, etc.)."""
    d = {f: getattr(w, f) for f in w.__dataclass_fields__}
    d.update(kw)
    return Workload(**d)


def layer_bytes(w: Workload) -> int:
    """Bytes of one layer's expert weights."""
    es = 2 if w.act == "bf16" else 4
    return 3 * w.E * w.F * w.d * es


def flops_per_token(w: Workload) -> int:
    """Expert FLOPs per token: K * 6 * d * F."""
    return w.K * 6 * w.d * w.F


def checksum(t: torch.Tensor) -> int:
    """64-bit order-dependent checksum of a tensor's raw bytes (for logging inputs)."""
    b = t.detach().contiguous().view(torch.uint8).reshape(-1).to("cpu").to(torch.int64)
    n = b.numel()
    wts = (torch.arange(n, dtype=torch.int64) % 251) + 1
    return int((b * wts).sum().item()) & ((1 << 64) - 1)

