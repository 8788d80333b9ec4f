"""The synthetic-input recipe: determinism, shapes, dtypes and the statistics it promises."""
import numpy as np
import torch

from oracle import r3_oracle as O
from paper_2510_11370_b200 import synth
from tests.helpers import Case, f64


def test_workload_table_matches_the_five_configurations():
    w = synth.WORKLOADS
    assert (w["c1_tiny_fp32"].T, w["c1_tiny_fp32"].d, w["c1_tiny_fp32"].E, w["c1_tiny_fp32"].K,
            w["c1_tiny_fp32"].F, w["c1_tiny_fp32"].act) == (512, 128, 8, 2, 256, "f32")
    for name, T in [("c2_layer_bf16", 4096), ("c3_skewed", 32768), ("c4_replay", 65536),
                    ("c5_stack48", 16384)]:
        c = w[name]
        assert (c.T, c.d, c.E, c.K, c.F, c.act) == (T, 2048, 128, 8, 768, "bf16")
    assert w["c4_capture"].layers == 48 and w["c4_capture"].T == 256
    assert w["c4_capture"].router_w == "bf16" and w["c4_capture"].idx_dtype == torch.uint8
    assert w["c5_stack48"].layers == 48
    assert synth.layer_bytes(w["c2_layer_bf16"]) == 1_207_959_552
    assert synth.flops_per_token(w["c2_layer_bf16"]) == 75_497_472


def test_tensors_are_deterministic_and_distributed_as_stated():
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], T=256, E=8, F=64, d=256)
    a, b = synth.activations(w), synth.activations(w)
    assert torch.equal(a, b) and a.dtype == torch.bfloat16 and a.shape == (256, 256)
    assert abs(a.float().std().item() - 1.0) < 0.05
    wg, wu, wd = synth.expert_weights(w)
    assert wg.shape == (8, 64, 256) and wd.shape == (8, 256, 64)
    assert abs(wg.float().std().item() - 0.02) < 0.002
    assert synth.router_weight(w).dtype == torch.float32
    assert not torch.equal(synth.activations(w, layer=1), a)
    assert synth.checksum(a) == synth.checksum(b)


def test_resampled_record_changes_about_ten_percent_of_tokens_by_one_expert():
    case = Case(synth.WORKLOADS["c1_tiny_fp32"])
    own = O.topk_indices(case.s, 2)
    rec = case.idx_np()
    O.check_record(rec, 8)
    diff = (own != rec).sum(axis=1)
    assert set(np.unique(diff)) <= {0, 1}
    assert 0.05 < (diff > 0).mean() < 0.16


def test_drifted_record_is_valid_and_differs_at_the_paper_like_rate():
    w = synth.scaled(synth.WORKLOADS["c2_layer_bf16"], T=512, F=64)
    x, w_r = synth.activations(w), synth.router_weight(w)
    s = O.router_logits(f64(x), f64(w_r))
    rec = synth.make_record(w, torch.from_numpy(s)).to(torch.int64).numpy()
    O.check_record(rec, w.E)
    own = O.topk_indices(s, w.K)
    differing = np.mean([len(set(a) - set(b)) for a, b in zip(own, rec)]) / w.K
    assert 0.02 < differing < 0.25     # Section 3.2: about one routed expert in ten differs


def test_zipf_bias_skews_the_record():
    w = synth.scaled(synth.WORKLOADS["c3_skewed"], T=2048, F=64)
    x, w_r = synth.activations(w), synth.router_weight(w)
    s = O.router_logits(f64(x), f64(w_r))
    rec = synth.make_record(w, torch.from_numpy(s)).to(torch.int64).numpy()
    O.check_record(rec, w.E)
    counts = np.bincount(rec.reshape(-1), minlength=w.E)
    assert counts.max() > 0.9 * w.T and (counts == 0).sum() + (counts < 8).sum() > 20
    bias = synth.zipf_bias(w)
    assert bias.max().item() == 0.0 and abs(bias.min().item() + 1.2 * np.log(128)) < 1e-5
