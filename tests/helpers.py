"""Shared test helpers: build a synthetic case on the CPU, widen it for the oracle."""
import numpy as np
import torch

from oracle import r3_oracle as O
from paper_2510_11370_b200 import synth


def f64(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a stored tensor (bf16 / f32) to float64 numpy."""
    return t.detach().to("cpu").to(torch.float64).numpy()


def f32(t: torch.Tensor) -> np.ndarray:
    """Exact widening of a stored tensor (bf16 / f32) to float32 numpy (halves oracle memory)."""
    return t.detach().to("cpu").to(torch.float32).numpy()


class Case:
    """Inputs of one replayed layer (CPU tensors) plus the oracle's logits and the record."""

    def __init__(self, w: synth.Workload, layer: int = 0, device="cpu"):
        self.w = w
        self.x = synth.activations(w, device, layer).cpu()
        self.dy = synth.upstream_grad(w, device, layer).cpu()
        self.w_r = synth.router_weight(w, device, layer).cpu()
        self.w_gate, self.w_up, self.w_down = (t.cpu() for t in synth.expert_weights(w, device, layer))
        self.s = O.router_logits(f64(self.x), f64(self.w_r))
        self.idx = synth.make_record(w, torch.from_numpy(self.s), layer).cpu()

    def idx_np(self) -> np.ndarray:
        return self.idx.to(torch.int64).numpy()

    def oracle_layer(self):
        return O.layer_fwd_bwd(f64(self.x), f64(self.w_r), self.idx_np(), f32(self.w_gate),
                               f32(self.w_up), f32(self.w_down), f64(self.dy))

    def cuda(self):
        return {k: getattr(self, k).cuda() for k in
                ("x", "dy", "w_r", "w_gate", "w_up", "w_down", "idx")}


def rel_err(got, ref) -> float:
    """max |err| / max |ref| - the tolerance measure of the benchmark brief."""
    got = np.asarray(got, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    denom = np.abs(ref).max()
    return float(np.abs(got - ref).max() / (denom if denom > 0 else 1.0))


def random_record(rng: np.random.Generator, T: int, E: int, K: int, dtype) -> torch.Tensor:
    """K distinct experts per token, uniformly random, random slot order."""
    keys = rng.random((T, E))
    idx = np.argsort(keys, axis=1)[:, :K]
    return torch.from_numpy(idx.astype(np.int64)).to(dtype)
