#!/usr/bin/env python
"""Benchmark of the replayed-routing MoE layer (forward + router-logit backward) on B200.

    python bench.py --gpus 1 --steps 20 --warmup 5                 # this library, every config
    python bench.py --workload c2_layer_bf16 --steps 1000          # one configuration alone
    python bench.py --impl reference --steps 2 --warmup 1          # the CPU oracle, timed
    python bench.py --gpus 2 ...                                   # starts 2 ranks itself
    python -m torch.distributed.run --nproc-per-node N ... bench.py --gpus N ...

A step is one pass of the whole path over one synthetic batch: training logits, replay gate,
permute, grouped SwiGLU experts, combine, dgates, dlogits (the last four steps of the layer run as
one kernel; the per-kernel table also times the separate entry points).  The headline workload is
the largest single-layer configuration, the replay of a recorded 65536-token batch (c4_replay);
with one GPU and no --workload the line also carries `per_config`: the same measurement for the
tiny fp32 layer, the 4096-token layer, the skewed 32768-token layer, the 48-layer decode capture,
the 65536-token replay and the 48-block stack.  One JSON line is printed by rank 0.
"""
from __future__ import annotations

import argparse
import ctypes
import json
import math
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "replayed-MoE-layer tokens/s (fwd+router bwd)"
UNIT = "tokens/s"
HEADLINE = "c4_replay"
L2_BYTES = 126e6
SUSTAINED_SECONDS = 0.6
NOMINAL_HBM_GBS = 8000.0
NOMINAL_BF16_TFLOPS = 2250.0
# DRAM bytes of one router_pair_kernel launch on the 48 x 256 decode capture (75.6 MB read +
# 1.5 MB written; algorithmic 75.6 MB), from the ncu capture of that workload.
CAPTURE_DRAM_TRAFFIC_BYTES = 77.05e6
# DRAM bytes (read + write) of one launch of the up-projection GEMM kernel, from the ncu captures
# summarised under profiles/ (a constant taken from the profile, not re-measured by a run)
GEMM_UP_DRAM_TRAFFIC_BYTES = {"c2_layer_bf16": 988.8e6,     # 940.8 MB read + 48.0 MB written
                              "c4_replay": 3.742e9}         # 2.95 GB read + 791.8 MB written


def launches_per_step(w) -> int:
    """Kernel launches of one r3_replay_layer call on workload w (all of them this library's)."""
    bf16 = w.act == "bf16"
    router_tc = bf16 and w.E % 16 == 0 and w.E <= 256 and w.K <= 16
    n = 1                                   # router logits
    if router_tc and w.router_w == "f32":
        n += 1                              # float32 router weights split into three bf16 planes
    n += 2                                  # dispatch maps (one cluster / cooperative launch), row copy
    if not bf16 or w.T > 4096:
        n += 1                              # work lists (up to 4096 tokens the dispatch builds them)
    n += 2                                  # the two expert GEMMs
    n += 1 if w.K <= 8 else 4               # finish: gate + combine + dgates + dlogits in one pass
    return n


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            p = json.load(f)
        return dict(hbm_gbs=float(p["hbm_gbs"]), bf16_tflops=float(p["bf16_tflops"]),
                    bf16_tflops_sustained=float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                    source="measured")
    return dict(hbm_gbs=6650.0, bf16_tflops=1590.0, bf16_tflops_sustained=1400.0,
                source="fallback")


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi for the whole run; a timed region
    asks for the samples that fell inside its wall-clock window."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index = index
        self.rows = []
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.FIELDS}",
                 "--format=csv,noheader,nounits", "-lms", "50"],
                stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except OSError:
            self.proc = None
            return self
        threading.Thread(target=self._read, daemon=True).start()
        time.sleep(0.3)
        return self

    def _read(self):
        for line in self.proc.stdout:
            self.rows.append((time.time(), [c.strip() for c in line.split(",")]))

    def stop(self):
        if self.proc is None:
            return
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except subprocess.TimeoutExpired:
            self.proc.kill()
        self.proc = None

    def window(self, t0: float, t1: float) -> dict:
        """Clock record of the wall-clock window [t0, t1] (a region shorter than the sampling
        period takes the nearest samples around it)."""
        empty = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return empty
        if time.time() < t1 + 0.12:
            time.sleep(0.12)
        good = [(ts, r) for (ts, r) in list(self.rows) if len(r) >= 7]
        rows = [r for (ts, r) in good if t0 <= ts <= t1 + 0.02]
        if not rows:
            rows = [r for (ts, r) in good if t0 - 0.06 <= ts <= t1 + 0.1]
        if not rows:
            return empty

        def num(v):
            try:
                return float(v)
            except ValueError:
                return None
        sm = [num(r[0]) for r in rows if num(r[0]) is not None]
        reasons = [n for i, n in enumerate(self.NAMES)
                   if any(r[3 + i].lower() == "active" for r in rows)]
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": num(rows[0][1]),
                "power_w_max": max((num(r[2]) or 0) for r in rows), "reasons": reasons,
                "samples": len(rows)}


def clocks_max_mhz():
    """Maximum SM clock of GPU 0 as nvidia-smi states it (None when it cannot be read)."""
    try:
        out = subprocess.run(["nvidia-smi", "--query-gpu=clocks.max.sm", "--format=csv,noheader,nounits",
                              "-i", "0"], capture_output=True, text=True, timeout=10).stdout
        return float(out.strip().splitlines()[0])
    except Exception:
        return None


def layer_config(w, tokens_per_gpu=None) -> dict:
    """The `config` object of a one-layer workload; both arms print exactly this."""
    from paper_2510_11370_b200 import synth
    return {"workload": w.name, "T": w.T, "d": w.d, "E": w.E, "K": w.K, "F": w.F,
            "router": "fp32 logits/softmax, %s router weights" % w.router_w,
            "tokens_per_gpu": tokens_per_gpu or w.T, "streams": 2,
            "l2": "inputs larger than L2: %.2f GB of expert weights and %.2f GB of grouped rows "
                  "stream through the 126 MB L2 every step"
                  % (synth.layer_bytes(w) / 1e9, 2.0 * w.T * w.K * w.d * (2 if w.act == "bf16" else 4) / 1e9)
                  if synth.layer_bytes(w) > 2 * L2_BYTES else
                  "working set below L2 (a correctness configuration): warm-L2 numbers"}


# ---------------------------------------------------------------------------------------------
# the CPU oracle, timed (cpu_baseline leg and --impl reference)
# ---------------------------------------------------------------------------------------------
def oracle_inputs(w, n_tokens, tensors=None):
    """Oracle inputs for the first n_tokens of the workload with all experts' weights: from the
    given device tensors (x, dy, w_r, wg, wu, wd) when the GPU arm already holds them, else drawn
    on the CPU by the same recipe."""
    import torch
    from paper_2510_11370_b200 import synth
    from oracle import r3_oracle as O
    if tensors is None:
        x = synth.activations(w, "cpu")[:n_tokens]
        dy = synth.upstream_grad(w, "cpu")[:n_tokens]
        w_r = synth.router_weight(w, "cpu")
        wg, wu, wd = synth.expert_weights(w, "cpu")
    else:
        x, dy = tensors[0][:n_tokens].cpu(), tensors[1][:n_tokens].cpu()
        w_r, wg, wu, wd = (t.cpu() for t in tensors[2:])
    f64 = lambda t: t.to(torch.float64).numpy()
    f32 = lambda t: t.to(torch.float32).numpy()
    s = O.router_logits(f64(x), f64(w_r))
    wn = synth.scaled(w, T=n_tokens)
    idx = synth.make_record(wn, torch.from_numpy(s)).to(torch.int64).numpy()
    return dict(x=f64(x), dy=f64(dy), w_r=f64(w_r), wg=f32(wg), wu=f32(wu), wd=f32(wd), idx=idx)


def oracle_step(inp):
    from oracle import r3_oracle as O
    return O.layer_fwd_bwd(inp["x"], inp["w_r"], inp["idx"], inp["wg"], inp["wu"], inp["wd"],
                           inp["dy"])


def blas_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def time_oracle(inp, n_tokens, steps, warmup, min_seconds=0.0, max_steps=40):
    """Times the oracle on prepared inputs; with min_seconds it keeps adding passes (at most
    max_steps) until that much CPU time is spent.  Returns (tokens/s, seconds per pass, passes)."""
    for _ in range(warmup):
        oracle_step(inp)
    t0 = time.perf_counter()
    done = 0
    while done < steps or (time.perf_counter() - t0 < min_seconds and done < max_steps):
        oracle_step(inp)
        done += 1
    dt = (time.perf_counter() - t0) / max(done, 1)
    return n_tokens / dt, dt, done


def run_reference(args, w):
    """The oracle as it stands on the host cores: each step is the whole layer (forward +
    router-logit backward, float64 numpy) on a bounded sample of the workload's tokens."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    n = min(w.T, args.ref_tokens)
    inp = oracle_inputs(w, n)
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    # one calibration pass bounds the whole run to a few minutes
    t0 = time.perf_counter()
    oracle_step(inp)
    t_one = time.perf_counter() - t0
    budget = 150.0
    if (steps + warmup) * t_one > budget:
        warmup = min(warmup, 1)
        steps = max(1, min(steps, int(budget / t_one) - warmup))
    tps, dt, _ = time_oracle(inp, n, steps, warmup)
    sample = (f"tokens [0,{n}) of {w.name} (all {w.E} experts' weights), whole layer fwd + "
              f"router-logit bwd in float64 numpy, {steps} timed step(s) after {warmup} warm-up")
    line = {
        "impl": "reference", "metric": METRIC, "value": tps, "unit": UNIT, "n_gpus": args.gpus,
        "steps": steps, "warmup": warmup, "ms_per_step": dt * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": layer_config(w),
        "cpu_baseline": {"value": tps, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": tps, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------
# timing helpers
# ---------------------------------------------------------------------------------------------
def event_time(torch, fn, n):
    """Average milliseconds of n calls of fn(i) between two CUDA events on the current stream."""
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for i in range(n):
        fn(i)
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / n


def sustained_region(torch, sampler, step, ms_guess, units_per_step, seconds=SUSTAINED_SECONDS):
    """The same step repeated for at least `seconds`: milliseconds per step under whatever clock
    the power cap allows, the median sampled SM clock, and time x clock beside it."""
    n = max(3, int(math.ceil(seconds * 1e3 / max(ms_guess, 1e-3))))
    t0 = time.time()
    ms = event_time(torch, lambda i: step(), n)
    t1 = time.time()
    clk = sampler.window(t0, t1) if sampler else {"sm_mhz": None, "reasons": [], "samples": 0}
    out = {"ms_per_step": ms, "value": units_per_step / (ms * 1e-3), "steps": n,
           "seconds": round(ms * n * 1e-3, 3), "clocks": clk}
    if clk.get("sm_mhz"):
        out["ms_x_sm_mhz"] = round(ms * clk["sm_mhz"], 2)
    return out


def ring_count(bytes_per_call: float) -> int:
    """How many argument sets a kernel's timing loop rotates over, so that a set has left the L2
    before it is used again (a call that itself streams more than twice the L2 needs one)."""
    return max(1, min(160, int(math.ceil(2.0 * L2_BYTES / max(bytes_per_call, 1.0)))))


def tensor_roofline(peaks, achieved, flop, algo_bytes, long_run, kernel, traffic=None):
    """Roofline object of a tensor-core kernel: achieved TFLOP/s against the measured cuBLAS
    figure (sustained for a region of a quarter second or more, else burst) and against the
    binding roof min(tensor peak, arithmetic intensity x measured copy bandwidth)."""
    peak = peaks["bf16_tflops_sustained"] if long_run else peaks["bf16_tflops"]
    ai = flop / algo_bytes
    hbm_roof = ai * peaks["hbm_gbs"] / 1e3                     # TFLOP/s
    bound = min(peak, hbm_roof)
    return {"bound": "tensor", "kernel": kernel, "achieved": round(achieved, 2), "peak": peak,
            "unit": "TFLOP/s", "frac": round(achieved / peak, 4),
            "peak_kind": f"bf16 matmul {'sustained' if long_run else 'burst'}, {peaks['source']}",
            "frac_of_burst": round(achieved / peaks["bf16_tflops"], 4),
            "frac_of_sustained": round(achieved / peaks["bf16_tflops_sustained"], 4),
            "frac_of_nominal_2250": round(achieved / NOMINAL_BF16_TFLOPS, 4),
            "flop_per_byte": round(ai, 1), "hbm_roof_tflops": round(hbm_roof, 1),
            "min_bound": "hbm" if hbm_roof < peak else "tensor",
            "frac_of_min_bound": round(achieved / bound, 4),
            "traffic": traffic,
            "traffic_source": "ncu capture summarised under profiles/ (a constant, not re-measured "
                              "by this run)" if traffic else None}


# ---------------------------------------------------------------------------------------------
# one replayed layer (configs 1, 2, 3, 4-replay)
# ---------------------------------------------------------------------------------------------
class LayerInputs:
    """Seeded inputs of one layer workload on the device (rank-dependent seed)."""

    def __init__(self, torch, r3, synth, w, dev, rank=0):
        self.w = wk = synth.scaled(w, seed=w.seed + rank)
        self.s = r3.shape_of(wk)
        self.x = synth.activations(wk, dev)
        self.dy = synth.upstream_grad(wk, dev)
        self.w_r = synth.router_weight(wk, dev)
        self.wg, self.wu, self.wd = synth.expert_weights(wk, dev)
        _, logits0 = r3.capture_topk_ws(self.s, 1, self.x, self.w_r, want_idx=False, want_logits=True)
        # inference-side record emulated from drifted logits (the library's own logits: nothing of
        # the oracle enters the product path)
        self.idx = synth.make_record(wk, logits0)


def checksum(torch, t):
    """64-bit wrap-around sum of the tensor's raw 16/32/8-bit words."""
    raw = t.contiguous().view(torch.int16 if t.element_size() == 2 else
                              torch.int32 if t.element_size() == 4 else torch.uint8).reshape(-1)
    total = 0
    for lo in range(0, raw.numel(), 1 << 27):
        total += int(raw[lo:lo + (1 << 27)].to(torch.int64).sum().item())
    return total & ((1 << 64) - 1)


def measure_layer(torch, r3, r3dist, inp, args, peaks, sampler, world=1, dev=None, *,
                  detail=True, e2e=False):
    """Times the whole path on one layer workload.  Returns the record of that configuration."""
    wk, s = inp.w, inp.s
    x, dy, w_r, wg, wu, wd, idx = inp.x, inp.dy, inp.w_r, inp.wg, inp.wu, inp.wd, inp.idx
    T, K, E, d, F = wk.T, wk.K, wk.E, wk.d, wk.F
    R = T * K
    es = 2 if wk.act == "bf16" else 4
    steps, warmup = args.steps, max(args.warmup, 3)

    st = r3.new_status(dev)
    y = torch.empty((T, d), dtype=wk.act_dtype, device=dev)
    dlogits = torch.empty((T, E), dtype=torch.float32, device=dev)
    gates = torch.empty((T, K), dtype=torch.float32, device=dev)
    ws = r3.workspace(r3.replay_layer_workspace_bytes(s), dev)

    def step():
        r3.replay_layer(s, x, w_r, idx, wg, wu, wd, dy, y=y, dlogits=dlogits, gates=gates, ws=ws,
                        dev_status=st)

    # ---- whole-path throughput, inputs resident in HBM: exactly `steps` steps ------------------
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    r3dist.barrier()
    torch.cuda.synchronize()
    t_wall0 = time.time()
    ev0.record()
    for _ in range(steps):
        step()
    ev1.record()
    torch.cuda.synchronize()
    r3dist.barrier()
    t_wall1 = time.time()
    ms_total = r3dist.max_over_ranks(ev0.elapsed_time(ev1), dev)
    assert st.item() == 0, f"device status {st.item()}"
    ms_per_step = ms_total / steps
    rec = {"workload": wk.name, "ms_per_step": ms_per_step,
           "value": world * T * steps / (ms_total * 1e-3), "unit": UNIT, "steps": steps,
           "warmup": warmup, "timed_ms": ms_total,
           "config": layer_config(wk), "gpu_launches": launches_per_step(wk) * steps,
           "clocks": sampler.window(t_wall0, t_wall1) if sampler else None}

    if not detail:
        if not args.no_sustained:
            rec["sustained"] = sustained_region(torch, sampler, step, ms_per_step, T)
        return rec

    # ---- the same step timed one by one: best and median ---------------------------------------
    n_single = min(max(steps, 20), 100)
    single = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
              for _ in range(n_single)]
    for a, b in single:
        a.record()
        step()
        b.record()
    torch.cuda.synchronize()
    single_ms = sorted(a.elapsed_time(b) for a, b in single)
    rec["per_step"] = {"best_ms": round(single_ms[0], 5),
                       "median_ms": round(statistics.median(single_ms), 5), "steps": n_single}

    # ---- per-kernel segments in the layer's own order (events between the entry points) ---------
    seg_names = ["logits", "permute", "expert_up_swiglu", "expert_down", "finish_fused"]
    logits = torch.empty((T, E), dtype=torch.float32, device=dev)
    dg = torch.empty((T, K), dtype=torch.float32, device=dev)
    pout = (torch.empty(E, dtype=torch.int32, device=dev),
            torch.empty(E + 1, dtype=torch.int32, device=dev),
            torch.empty((T, K), dtype=torch.int32, device=dev),
            torch.empty(R, dtype=torch.int32, device=dev),
            torch.empty((R, d), dtype=wk.act_dtype, device=dev))
    o = torch.empty((R, d), dtype=wk.act_dtype, device=dev)
    pws = r3.workspace(r3.permute_workspace_bytes(s), dev)
    gws = r3.workspace(r3.grouped_swiglu_workspace_bytes(s), dev)
    rws = r3.workspace(r3.capture_topk_workspace_bytes(s, 1), dev)
    fused = K <= 8
    seg_steps = min(max(steps, 5), 20)
    evs = [[torch.cuda.Event(enable_timing=True) for _ in range(len(seg_names) + 1)]
           for _ in range(seg_steps)]

    def finish():
        if fused:
            r3.replay_finish(s, logits, idx, o, pout[2], dy, y=y, gates=gates, dlogits=dlogits,
                             dev_status=st)
        else:
            r3.replay_gate_fwd(s, logits, idx, gates=gates, dev_status=st)
            r3.combine(s, o, pout[2], gates, y=y)
            r3.combine_bwd_gates(s, dy, o, pout[2], dgates=dg)
            r3.replay_gate_bwd(s, gates, dg, idx, dlogits=dlogits)

    def seg_step(e):
        e[0].record()
        r3.capture_topk_ws(s, 1, x, w_r, logits_out=logits, want_idx=False, ws=rws)
        e[1].record()
        r3.permute(s, idx, x, out=pout, ws=pws, dev_status=st)
        e[2].record()
        r3.expert_up_swiglu(s, pout[4], pout[1], wg, wu, gws, dev_status=st)
        e[3].record()
        r3.expert_down(s, wd, o, gws, dev_status=st)
        e[4].record()
        finish()
        e[5].record()

    for _ in range(3):
        seg_step(evs[0])
    torch.cuda.synchronize()
    t_seg0 = time.time()
    for e in evs:
        seg_step(e)
    torch.cuda.synchronize()
    t_seg1 = time.time()
    seg_ms = {n: statistics.mean(e[i].elapsed_time(e[i + 1]) for e in evs)
              for i, n in enumerate(seg_names)}
    flops = {"expert_up_swiglu": 4.0 * R * d * F, "expert_down": 2.0 * R * d * F,
             "logits": 2.0 * T * d * E}
    rw = 2 if wk.router_w == "bf16" else 4
    algo_bytes = {                                  # algorithmic bytes per call
        "logits": T * d * es + E * d * rw + T * E * 4,
        "gate_fwd": T * (E * 4 + K * 1 + K * 4),
        "permute": T * (K + d * es + K * 8 + K * d * es),
        "permute_maps": T * (K + K * 8),
        "combine": T * (K * d * es + K * 8 + d * es),
        "dgates": T * (d * es + K * d * es + K * 4 + K * 4),
        "gate_bwd": T * (K * 9 + E * 4),
        "finish_fused": T * (K * d * es + 2 * d * es + K * 9 + K * 4 + E * 4),
        "expert_up_swiglu": 2 * E * F * d * es + R * d * es + R * F * es,
        "expert_down": E * F * d * es + R * F * es + R * d * es,
    }
    kernels = {n: {"ms_in_sequence": round(seg_ms[n], 5)} for n in seg_names}
    for n in ("expert_up_swiglu", "expert_down", "logits"):
        kernels[n]["tflops"] = round(flops[n] / (seg_ms[n] * 1e-3) / 1e12, 1)

    # ---- the memory-bound kernels one by one, each over a ring of argument sets larger than L2 -
    def clones(t, n):
        return [t] + [t.clone() for _ in range(n - 1)]

    def ring_time(name, nbytes, make, call):
        """make(n) -> list of n argument sets; call(set) runs the kernel once."""
        n = ring_count(nbytes)
        sets = make(n)
        reps = max(2 * n, 20) if nbytes < 50e6 else max(n, 10)
        for i in range(n):
            call(sets[i])
        torch.cuda.synchronize()
        ms = event_time(torch, lambda i: call(sets[i % n]), reps)
        gbs = nbytes / (ms * 1e-3) / 1e9
        kernels.setdefault(name, {}).update(
            {"ms": round(ms, 5), "hbm_gbs": round(gbs, 1),
             "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 3),
             "frac_of_nominal_8tbs": round(gbs / NOMINAL_HBM_GBS, 3),
             "l2": f"ring of {n} argument set(s), {n * nbytes / 1e6:.0f} MB in all"})
        del sets
        return ms

    ring_time("logits", algo_bytes["logits"],
              lambda n: list(zip(clones(x, n), clones(logits, n))),
              lambda a: r3.capture_topk_ws(s, 1, a[0], w_r, logits_out=a[1], want_idx=False, ws=rws))
    ring_time("gate_fwd", algo_bytes["gate_fwd"],
              lambda n: list(zip(clones(logits, n), clones(idx, n), clones(gates, n))),
              lambda a: r3.replay_gate_fwd(s, a[0], a[1], gates=a[2], dev_status=st))
    ring_time("gate_bwd", algo_bytes["gate_bwd"],
              lambda n: list(zip(clones(gates, n), clones(dg, n), clones(idx, n), clones(dlogits, n))),
              lambda a: r3.replay_gate_bwd(s, a[0], a[1], a[2], dlogits=a[3]))
    ring_time("permute_maps", algo_bytes["permute_maps"],
              lambda n: list(zip(clones(idx, n), clones(pout[2], n), clones(pout[3], n))),
              lambda a: r3.permute(s, a[0], None, out=(pout[0], pout[1], a[1], a[2], None), ws=pws,
                                   dev_status=st))
    ms_perm = ring_time("permute", algo_bytes["permute"],
                        lambda n: list(zip(clones(idx, n), clones(x, n), clones(pout[4], n))),
                        lambda a: r3.permute(s, a[0], a[1], out=pout[:4] + (a[2],), ws=pws,
                                             dev_status=st))
    # the row copy alone: the dispatch with rows minus the maps-only dispatch
    rows_ms = ms_perm - kernels["permute_maps"]["ms"]
    if rows_ms > 0:
        rows_gbs = T * (d * es + K * 4 + K * d * es) / (rows_ms * 1e-3) / 1e9
        kernels["permute_rows"] = {"ms": round(rows_ms, 5), "hbm_gbs": round(rows_gbs, 1),
                                   "frac_of_measured_hbm": round(rows_gbs / peaks["hbm_gbs"], 3),
                                   "derived": "permute - permute_maps"}
    ring_time("combine", algo_bytes["combine"],
              lambda n: list(zip(clones(o, n), clones(y, n))),
              lambda a: r3.combine(s, a[0], pout[2], gates, y=a[1]))
    ring_time("dgates", algo_bytes["dgates"],
              lambda n: list(zip(clones(o, n), clones(dy, n))),
              lambda a: r3.combine_bwd_gates(s, a[1], a[0], pout[2], dgates=dg))
    if fused:
        # what r3_replay_layer runs instead of gate_fwd + combine + dgates + gate_bwd (K <= 8)
        ring_time("finish_fused", algo_bytes["finish_fused"],
                  lambda n: list(zip(clones(o, n), clones(dy, n), clones(y, n), clones(dlogits, n),
                                     clones(logits, n))),
                  lambda a: r3.replay_finish(s, a[4], idx, a[0], pout[2], a[1], y=a[2], gates=gates,
                                             dlogits=a[3], dev_status=st))
    assert st.item() == 0
    rec["kernels"] = kernels

    # ---- roofline of the dominant kernel: the up-projection grouped GEMM -----------------------
    achieved = flops["expert_up_swiglu"] / (seg_ms["expert_up_swiglu"] * 1e-3) / 1e12
    if wk.act == "bf16":
        long_run = (t_seg1 - t_seg0) >= 0.25
        rec["roofline"] = tensor_roofline(
            peaks, achieved, flops["expert_up_swiglu"], algo_bytes["expert_up_swiglu"], long_run,
            "grouped_gemm_pair_kernel<0> (gate/up + SwiGLU); its events bracket the "
            "r3_expert_up_swiglu call, which also holds the one-CTA work-list kernel",
            GEMM_UP_DRAM_TRAFFIC_BYTES.get(wk.name))
        down = flops["expert_down"] / (seg_ms["expert_down"] * 1e-3) / 1e12
        rec["roofline_down"] = tensor_roofline(
            peaks, down, flops["expert_down"], algo_bytes["expert_down"], long_run,
            "grouped_gemm_pair_kernel<1> (down projection)")
    else:
        # float32 activations run the plain-FMA grouped GEMM (tf32 would break the 1e-5 bar):
        # 148 SMs x 128 FMA lanes x 2 FLOP at the maximum SM clock
        alu_peak = 148 * 128 * 2 * (clocks_max_mhz() or 1965.0) * 1e6 / 1e12
        rec["roofline"] = {"bound": "alu", "kernel": "simt_grouped_gemm_kernel (gate/up + SwiGLU, float32)",
                           "achieved": round(achieved, 2), "peak": round(alu_peak, 1),
                           "unit": "TFLOP/s", "frac": round(achieved / alu_peak, 4),
                           "peak_kind": "fp32 FMA: 148 SMs x 128 lanes x 2 x max SM clock",
                           "traffic": None}
    del o, pout, logits
    # ---- the same step for at least SUSTAINED_SECONDS (power-capped clocks).  It comes after the
    # per-kernel timings, so that those, like the K timed steps, are taken before the long region
    # has driven the GPU into its power cap (their peak is the burst figure) ----------------------
    if not args.no_sustained:
        rec["sustained"] = sustained_region(torch, sampler, step, ms_per_step, T)
    assert st.item() == 0
    if not e2e:
        return rec

    # ---- a second pass over the same record (the Update stage after the Recompute stage) -------
    step()
    y_first = y.clone()
    sr_steps = min(steps, 50)

    def again():
        r3.replay_layer_same_record(s, x, w_r, idx, wg, wu, wd, dy, y=y, dlogits=dlogits,
                                    gates=gates, ws=ws, dev_status=st)
    for _ in range(3):
        again()
    torch.cuda.synchronize()
    ms_sr = event_time(torch, lambda i: again(), sr_steps)
    assert torch.equal(y, y_first), "second pass over the record disagrees with the first"
    rec["same_record_pass"] = {"ms_per_step": round(ms_sr, 5), "steps": sr_steps,
                               "launches_per_step": launches_per_step(wk) - 1
                               - (0 if wk.act == "bf16" and T <= 4096 else 1),   # no maps, no work lists
                               "note": "r3_replay_layer_same_record: dispatch maps and work lists of "
                                       "the preceding r3_replay_layer call used again; not the headline step"}

    # ---- end to end through the host-buffer entry point ----------------------------------------
    xh, dyh, idxh = (t.cpu().pin_memory() for t in (x, dy, idx))
    yh = torch.empty((T, d), dtype=wk.act_dtype).pin_memory()
    dlh = torch.empty((T, E), dtype=torch.float32).pin_memory()
    hws = r3.workspace(r3.replay_layer_host_workspace_bytes(s), dev)
    e2e_steps = min(steps, 20)
    for _ in range(3):
        r3.replay_layer_host(s, xh, w_r, idxh, wg, wu, wd, dyh, yh, dlh, ws=hws, dev_status=st)
    r3dist.barrier()
    torch.cuda.synchronize()
    ev0.record()
    for _ in range(e2e_steps):
        r3.replay_layer_host(s, xh, w_r, idxh, wg, wu, wd, dyh, yh, dlh, ws=hws, dev_status=st)
    ev1.record()
    torch.cuda.synchronize()
    r3dist.barrier()
    e2e_ms = r3dist.max_over_ranks(ev0.elapsed_time(ev1), dev)
    assert st.item() == 0
    # the host-buffer call sends a large batch through in chunks of tokens, whose router launches
    # may split d differently from the whole batch's: equal up to a bf16 rounding step
    y_dev, y_host = y.float(), yh.to(dev).float()
    assert float((y_host - y_dev).abs().max()) <= 2.0 ** -7 * float(y_dev.abs().max()), \
        "host-buffer path disagrees with the device path"
    del y_dev, y_host
    e2e_rec = {"value": world * T * e2e_steps / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(xh.numel() * es + dyh.numel() * es + idxh.numel() * idxh.element_size()),
               "d2h_bytes_per_step": int(yh.numel() * es + dlh.numel() * 4),
               "ms_per_step": e2e_ms / e2e_steps, "steps": e2e_steps}

    # the same with several batches in flight (r3_replay_layer_host_enqueue): every step still copies
    # its inputs in and its results out; the copies of one step run beside the kernels of another
    depth = int(os.environ.get("R3_BENCH_E2E_DEPTH", "2"))
    lanes = [dict(x=xh, dy=dyh, idx=idxh, y=yh, dl=dlh, ws=hws, stream=torch.cuda.Stream(device=dev))]
    for _ in range(depth - 1):
        lanes.append(dict(x=xh.clone().pin_memory(), dy=dyh.clone().pin_memory(),
                          idx=idxh.clone().pin_memory(),
                          y=torch.empty_like(yh).pin_memory(), dl=torch.empty_like(dlh).pin_memory(),
                          ws=r3.workspace(r3.replay_layer_host_workspace_bytes(s), dev),
                          stream=torch.cuda.Stream(device=dev)))
    torch.cuda.synchronize()

    def pipelined(n):
        for i in range(n):
            ln = lanes[i % depth]
            r3.replay_layer_host_enqueue(s, ln["x"], w_r, ln["idx"], wg, wu, wd, ln["dy"], ln["y"],
                                         ln["dl"], ws=ln["ws"], dev_status=st, stream=ln["stream"])
        for ln in lanes:
            ln["stream"].synchronize()

    pipelined(2 * depth)
    r3dist.barrier()
    torch.cuda.synchronize()
    tp0 = time.perf_counter()
    pipelined(e2e_steps)
    torch.cuda.synchronize()
    tp1 = time.perf_counter()
    r3dist.barrier()
    pipe_ms = r3dist.max_over_ranks((tp1 - tp0) * 1e3, dev)
    assert st.item() == 0
    # every lane ran the same chunked call as the single-batch measurement above: same bits
    assert all(torch.equal(ln["y"], yh) for ln in lanes)
    e2e_rec["batches_in_flight"] = {
        "depth": depth, "value": world * T * e2e_steps / (pipe_ms * 1e-3), "unit": UNIT,
        "ms_per_step": pipe_ms / e2e_steps, "steps": e2e_steps,
        "timing": "host clock around the enqueues and the synchronisation of every stream"}
    rec["e2e"] = e2e_rec
    return rec


# ---------------------------------------------------------------------------------------------
# config 4, inference side, and config 5
# ---------------------------------------------------------------------------------------------
def measure_capture(torch, r3, synth, w, args, peaks, sampler, dev):
    """Router logits + TopKMask of a decode batch for `w.layers` layers in one launch
    (r3_capture_topk_batched), records packed as uint8; inputs rotate over more than L2."""
    L, T, d, E, K = w.layers, w.T, w.d, w.E, w.K
    s = r3.shape_of(w)
    reps = 8                                  # rotate over > L2-sized rings: activations AND weights
    xs = [torch.stack([synth.activations(w, dev, l + 100 * r) for l in range(L)]) for r in range(reps)]
    wrs = [torch.stack([synth.router_weight(w, dev, l + 100 * r) for l in range(L)]) for r in range(reps)]
    idx = torch.empty((L, T, K), dtype=w.idx_dtype, device=dev)
    one_idx = torch.empty((T, K), dtype=w.idx_dtype, device=dev)
    steps, warmup = max(args.steps, 20), max(args.warmup, 3)

    def batched(i):
        r3.capture_topk_batched(s, L, xs[i % reps], wrs[i % reps], idx_out=idx)

    def one(i):
        r3.capture_topk(s, xs[i % reps][i % L], wrs[i % reps][i % L], idx_out=one_idx)

    for i in range(warmup):
        batched(i)
        one(i)
    torch.cuda.synchronize()
    t0 = time.time()
    ms_b = event_time(torch, batched, steps)
    t1 = time.time()
    ms_1 = event_time(torch, one, steps)
    n_sus = 3 if args.no_sustained else int(math.ceil(SUSTAINED_SECONDS * 1e3 / ms_b))
    ts0 = time.time()
    ms_sus = event_time(torch, batched, n_sus)
    ts1 = time.time()
    clk = sampler.window(ts0, ts1) if sampler else None
    bytes_b = L * (T * d * 2 + E * d * 2 + T * K)

    def kern(ms):
        gbs = bytes_b / ms / 1e6
        return {"ms": round(ms, 5), "hbm_gbs": round(gbs, 1),
                "frac_of_measured_hbm": round(gbs / peaks["hbm_gbs"], 3),
                "frac_of_nominal_8tbs": round(gbs / NOMINAL_HBM_GBS, 3)}
    sus = {"ms_per_step": ms_sus, "value": L * T / (ms_sus * 1e-3), "steps": n_sus,
           "seconds": round(ms_sus * n_sus * 1e-3, 3), "clocks": clk, "kernel": kern(ms_sus)}
    if clk and clk.get("sm_mhz"):
        sus["ms_x_sm_mhz"] = round(ms_sus * clk["sm_mhz"], 2)
    return {
        "workload": w.name, "metric": "capture layer-tokens/s (router logits + top-K -> uint8 record)",
        "value": L * T / (ms_b * 1e-3), "unit": "layer-tokens/s", "steps": steps, "warmup": warmup,
        "ms_per_step": ms_b, "dtype": "bf16",
        "config": {"workload": w.name, "layers": L, "T": T, "d": d, "E": E, "K": K,
                   "l2": f"activations and router weights rotate over {reps} sets of "
                         f"{L * (T + E) * d * 2 / 1e6:.0f} MB (> L2 in all)"},
        "roofline": {"bound": "hbm", "kernel": "router_pair_kernel (48 layers in one launch)",
                     "achieved": round(bytes_b / ms_b / 1e6, 1), "peak": peaks["hbm_gbs"],
                     "unit": "GB/s", "frac": round(bytes_b / ms_b / 1e6 / peaks["hbm_gbs"], 4),
                     "peak_kind": f"copy bandwidth, {peaks['source']}",
                     "traffic": CAPTURE_DRAM_TRAFFIC_BYTES if w.name == "c4_capture" else None,
                     "traffic_source": "ncu capture summarised under profiles/ (a constant, not "
                                       "re-measured by this run)"},
        "kernels": {"capture_batched": kern(ms_b),
                    "capture_one_layer": {"us_per_call": round(ms_1 * 1e3, 2)}},
        "record_bytes_per_step": L * T * K, "gpu_launches": steps,
        "clocks": sampler.window(t0, t1) if sampler else None, "sustained": sus,
    }


def measure_stack(torch, r3, synth, w, args, peaks, sampler, dev, train=False):
    """Config 5: `w.layers` MoE blocks back to back with all their weights resident
    (r3_replay_blocks; every block has its own seeded input, record and weights).  With train:
    the blocks chained through residual connections, forward and the exact backward chain
    (r3_replay_stack_train, expert-weight gradients left out: 116 GB of float32 for 48 blocks)."""
    L, T, d, E, K, F = w.layers, w.T, w.d, w.E, w.K, w.F
    s = r3.shape_of(w)
    x = torch.stack([synth.activations(w, dev, l) for l in range(L)])
    dy = torch.stack([synth.upstream_grad(w, dev, l) for l in range(L)])
    w_r = torch.stack([synth.router_weight(w, dev, l) for l in range(L)])
    wg = torch.empty((L, E, F, d), dtype=w.act_dtype, device=dev)
    wu = torch.empty((L, E, F, d), dtype=w.act_dtype, device=dev)
    wd = torch.empty((L, E, d, F), dtype=w.act_dtype, device=dev)
    idx = torch.empty((L, T, K), dtype=w.idx_dtype, device=dev)
    for l in range(L):
        a, b, c = synth.expert_weights(w, dev, l)
        wg[l], wu[l], wd[l] = a, b, c
        del a, b, c
        _, lg = r3.capture_topk_ws(s, 1, x[l], w_r[l], want_idx=False, want_logits=True)
        idx[l] = synth.make_record(w, lg, l)
    y = torch.empty_like(x)
    dl = torch.empty((L, T, E), dtype=torch.float32, device=dev)
    ws = r3.workspace(r3.replay_layer_workspace_bytes(s), dev)
    st = r3.new_status(dev)

    def step():
        r3.replay_blocks(s, L, x, w_r, idx, wg, wu, wd, dy, y=y, dlogits=dl, ws=ws, dev_status=st)

    if train:
        del y, ws
        tws = r3.workspace(r3.lib.r3_replay_stack_train_workspace_bytes(ctypes.byref(s), L), dev)

        def step():
            r3.replay_stack_train(s, L, x[0], w_r, idx, wg, wu, wd, dy[0], ws=tws, dev_status=st)

    steps, warmup = args.steps, max(args.warmup, 3)
    for _ in range(warmup):
        step()
    torch.cuda.synchronize()
    t0 = time.time()
    ms = event_time(torch, lambda i: step(), steps)
    t1 = time.time()
    assert st.item() == 0
    clocks = sampler.window(t0, t1) if sampler else None
    # forward 6 R d F per block; with train: forward, forward again, and the 12 R d F of the
    # two input-gradient products
    flop = (24.0 if train else 6.0) * T * K * d * F * L
    tf = flop / (ms * 1e-3) / 1e12
    per_block = launches_per_step(w)
    rec = {
        "workload": w.name, "value": T / (ms * 1e-3), "unit": UNIT, "steps": steps,
        "warmup": warmup, "ms_per_step": ms, "layer_tokens_per_s": L * T / (ms * 1e-3),
        "dtype": "bf16",
        "config": {"workload": w.name, "blocks": L, "T": T, "d": d, "E": E, "K": K, "F": F,
                   "mode": ("residual chain, forward + exact backward (dx, dlogits, dW_r; block "
                            "forward recomputed)" if train else "independent blocks, forward + "
                            "router backward"),
                   "weights_gb": round(3 * L * E * F * d * 2 / 1e9, 1), "streams": 2,
                   "l2": "58 GB of weights stream through the 126 MB L2 every step"},
        "roofline": {"bound": "tensor", "kernel": "both grouped GEMMs of all blocks (whole-step time, "
                     "all other kernels included)", "achieved": round(tf, 1),
                     "peak": peaks["bf16_tflops_sustained"], "unit": "TFLOP/s",
                     "frac": round(tf / peaks["bf16_tflops_sustained"], 4),
                     "frac_of_burst": round(tf / peaks["bf16_tflops"], 4),
                     "frac_of_nominal_2250": round(tf / NOMINAL_BF16_TFLOPS, 4),
                     "peak_kind": f"bf16 matmul sustained, {peaks['source']}", "traffic": None},
        # train: per block the forward, then the forward again plus 7 backward kernels
        # (scale_rows, build_work, two input-gradient GEMMs, swiglu_bwd, dx, dwr)
        "gpu_launches": (2 * per_block + 7 if train else per_block) * L * steps,
        "clocks": clocks,
    }
    total_s = ms * steps * 1e-3
    if total_s >= 0.5:
        rec["sustained"] = {"ms_per_step": ms, "value": T / (ms * 1e-3), "steps": steps,
                            "seconds": round(total_s, 3), "clocks": clocks,
                            "note": "the timed region itself is long enough"}
        if clocks and clocks.get("sm_mhz"):
            rec["sustained"]["ms_x_sm_mhz"] = round(ms * clocks["sm_mhz"], 2)
    else:
        rec["sustained"] = sustained_region(torch, sampler, step, ms, T)
    return rec


# ---------------------------------------------------------------------------------------------
def contract_line(rec, world, dtype, extra=None):
    """The one JSON line of the contract from a configuration's record."""
    line = {"metric": rec.get("metric", METRIC), "value": rec["value"], "unit": rec["unit"],
            "n_gpus": world, "steps": rec["steps"], "warmup": rec["warmup"],
            "ms_per_step": rec["ms_per_step"], "higher_is_better": True, "scaling": "weak",
            "vs_baseline": None, "dtype": dtype, "data": "synthetic"}
    for k in ("config", "roofline", "roofline_down", "cpu_baseline", "e2e", "gpu_launches", "clocks",
              "sustained", "per_step", "layer_tokens_per_s", "inputs", "kernels", "same_record_pass",
              "record_bytes_per_step"):
        if k in rec:
            line[k] = rec[k]
    if extra:
        line.update(extra)
    return line


def run_ours(args):
    """The headline workload (and, on one GPU without --workload, every configuration)."""
    import torch
    from paper_2510_11370_b200 import build, dist as r3dist, synth
    build.build()
    from paper_2510_11370_b200 import r3

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: there is no CPU path")
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    rank, world = r3dist.init("nccl")
    peaks = load_peaks()
    sampler = ClockSampler(local).start() if rank == 0 else None
    suite = args.workload == "all" and world == 1
    name = HEADLINE if args.workload == "all" else args.workload
    w = synth.WORKLOADS[name]
    per_config = {}

    def free():
        import gc
        gc.collect()
        torch.cuda.empty_cache()

    try:
        if w.layers > 1 and name == "c4_capture":
            rec = measure_capture(torch, r3, synth, w, args, peaks, sampler, dev)
        elif w.layers > 1:
            rec = measure_stack(torch, r3, synth, w, args, peaks, sampler, dev, train=args.train)
        else:
            inp = LayerInputs(torch, r3, synth, w, dev, rank)
            rec = measure_layer(torch, r3, r3dist, inp, args, peaks, sampler, world, dev,
                                detail=True, e2e=True)
            rec["inputs"] = {"torch": torch.__version__, "seed": inp.w.seed, "checksums": {
                k: checksum(torch, getattr(inp, a)) for k, a in
                (("x", "x"), ("dy", "dy"), ("w_router", "w_r"), ("w_gate", "wg"), ("w_up", "wu"),
                 ("w_down", "wd"), ("record", "idx"))}}
            # ---- the oracle on this machine's host cores (rank 0, single-GPU runs only) ------------
            if rank == 0 and world == 1 and not args.no_cpu_baseline:
                n = min(w.T, args.ref_tokens)
                oin = oracle_inputs(w, n, (inp.x, inp.dy, inp.w_r, inp.wg, inp.wu, inp.wd))
                tps, dt, passes = time_oracle(oin, n, 1, 0, min_seconds=10.0)
                del oin
                rec["cpu_baseline"] = {
                    "value": tps, "unit": UNIT, "cores": blas_threads(), "kind": "oracle",
                    "seconds": round(dt * passes, 2),
                    "sample": f"tokens [0,{n}) of {w.name} (all {w.E} experts' weights), whole "
                              f"layer fwd + router-logit bwd, float64 numpy, {passes} passes"}
            del inp
        free()
        if suite:
            for other in ("c1_tiny_fp32", "c2_layer_bf16", "c3_skewed", "c4_capture", HEADLINE,
                          "c5_stack48"):
                wo = synth.WORKLOADS[other]
                if other == HEADLINE:
                    r = {k: v for k, v in rec.items() if k not in ("inputs", "cpu_baseline")}
                elif other == "c4_capture":
                    r = measure_capture(torch, r3, synth, wo, args, peaks, sampler, dev)
                elif wo.layers > 1:
                    free_b, _ = torch.cuda.mem_get_info()
                    if free_b < 80e9:
                        r = {"workload": other, "skipped": "needs about 75 GB of free device memory"}
                    else:
                        r = measure_stack(torch, r3, synth, wo, args, peaks, sampler, dev)
                else:
                    inp = LayerInputs(torch, r3, synth, wo, dev, rank)
                    r = measure_layer(torch, r3, r3dist, inp, args, peaks, sampler, world, dev,
                                      detail=True, e2e=False)
                    del inp
                r["dtype"] = "f32" if wo.act != "bf16" else "bf16"
                per_config[other] = r
                free()
    finally:
        if sampler:
            sampler.stop()

    if rank == 0:
        extra = {"peaks": peaks}
        if suite:
            extra["per_config"] = per_config
        print(json.dumps(contract_line(rec, world, "bf16" if w.act == "bf16" else "f32", extra)),
              flush=True)
    if world > 1:
        torch.distributed.destroy_process_group()


def run_train(args, w):
    """Forward plus the whole Update-stage backward of one replayed layer (r3_replay_layer_train
    with expert-weight gradients), with the backward's pieces timed apart."""
    import torch
    from paper_2510_11370_b200 import build, synth
    build.build()
    from paper_2510_11370_b200 import r3
    if int(os.environ.get("RANK", "0")) != 0:
        return
    dev = torch.device("cuda", 0)
    peaks = load_peaks()
    s = r3.shape_of(w)
    T, K, E, d, F = w.T, w.K, w.E, w.d, w.F
    R = T * K
    x = synth.activations(w, dev)
    dy = synth.upstream_grad(w, dev)
    w_r = synth.router_weight(w, dev)
    wg, wu, wd = synth.expert_weights(w, dev)
    _, lg = r3.capture_topk_ws(s, 1, x, w_r, want_idx=False, want_logits=True)
    idx = synth.make_record(w, lg)
    st = r3.new_status(dev)
    ws = r3.workspace(r3.lib.r3_replay_layer_train_workspace_bytes(ctypes.byref(s)), dev)
    dws = (torch.empty((E, F, d), dtype=torch.float32, device=dev),
           torch.empty((E, F, d), dtype=torch.float32, device=dev),
           torch.empty((E, d, F), dtype=torch.float32, device=dev))

    def timed(fn, steps):
        for _ in range(3):
            fn()
        torch.cuda.synchronize()
        return event_time(torch, lambda i: fn(), steps)

    def step():
        r3.replay_layer_train(s, x, w_r, idx, wg, wu, wd, dy, ws=ws, dev_status=st,
                              expert_grads=True, dw_experts=dws)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(0).start()
    t0 = time.time()
    ms = timed(step, args.steps)
    t1 = time.time()
    clocks = sampler.window(t0, t1)
    sampler.stop()
    assert st.item() == 0
    # pieces
    counts, offsets, ros, sor, xp = r3.permute(s, idx, x)
    o, a, b = r3.grouped_swiglu_train(s, xp, offsets, wg, wu, wd)
    gates = torch.rand((T, K), dtype=torch.float32, device=dev)
    dout = torch.empty((R, d), dtype=w.act_dtype, device=dev)
    bws = r3.workspace(r3.lib.r3_grouped_swiglu_bwd_workspace_bytes(ctypes.byref(s)), dev)
    lws = r3.workspace(r3.replay_layer_workspace_bytes(s), dev)
    dl = torch.randn((T, E), dtype=torch.float32, device=dev)
    n = min(args.steps, 20)
    seg = {
        "forward": timed(lambda: r3.replay_layer(s, x, w_r, idx, wg, wu, wd, dy, ws=lws), n),
        "scale_rows": timed(lambda: r3.scale_rows(s, dy, gates, ros, dout), n),
        "dgrad": timed(lambda: r3.grouped_swiglu_bwd_input(s, dout, a, b, offsets, wg, wu, wd,
                                                           ws=bws), n),
        "dgrad_wgrad": timed(lambda: r3.grouped_swiglu_bwd(s, xp, dout, a, b, offsets, wg, wu, wd,
                                                           ws=bws), n),
        "input_grad_finish": timed(lambda: r3.input_grad_finish(s, dout, ros, sor, offsets, dl,
                                                                idx, x, w_r), n),
    }
    seg["wgrad"] = seg["dgrad_wgrad"] - seg["dgrad"]
    flop_fwd = 6.0 * R * d * F
    wgrad_bytes = 3.0 * E * F * d * 4 + 2.0 * R * d * 2 + 3.0 * R * F * 2
    line = {
        "metric": METRIC, "value": T / (ms * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "mode": "forward + backward (dx, dW_r, dW_experts)",
                   "T": T, "d": d, "E": E, "K": K, "F": F,
                   "l2": "weights (1.2 GB) and weight gradients (2.4 GB) exceed the 126 MB L2"},
        "segments_ms": {k: round(v, 4) for k, v in seg.items()},
        "tflops": {"step (18 R d F)": round(3 * flop_fwd / (ms * 1e-3) / 1e12, 1),
                   "dgrad": round(flop_fwd / (seg["dgrad"] * 1e-3) / 1e12, 1),
                   "wgrad": round(flop_fwd / (seg["wgrad"] * 1e-3) / 1e12, 1)},
        "wgrad_gbs": round(wgrad_bytes / (seg["wgrad"] * 1e-3) / 1e9, 1),
        "clocks": clocks, "peaks": peaks,
    }
    print(json.dumps(line), flush=True)


def run_ep(args, w):
    """Expert-parallel replayed layer (tokens AND experts split over the ranks): every rank holds
    E/N experts and routes w.T tokens of its own; two all-to-alls of rows per layer.  With one
    rank the collectives are still made (NCCL, world size 1)."""
    import torch
    import torch.distributed as dist
    from paper_2510_11370_b200 import build, dist as r3dist, synth
    build.build()
    from paper_2510_11370_b200 import r3
    from paper_2510_11370_b200.ep import (EpDirectRank, EpRank, PeerBuffers, ep_replay_layer,
                                          ep_replay_layer_direct)
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    rank, world = r3dist.env_rank_world()
    if not dist.is_initialized():
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        os.environ.setdefault("MASTER_PORT", "29533")
        dist.init_process_group("nccl", rank=rank, world_size=world, device_id=dev)
    peaks = load_peaks()
    wk = synth.scaled(w, seed=w.seed + rank)
    T, K, E, d, F = wk.T, wk.K, wk.E, wk.d, wk.F
    el = E // world
    x = synth.activations(wk, dev)
    dy = synth.upstream_grad(wk, dev)
    w_r = synth.router_weight(w, dev)                    # replicated: same seed on every rank
    wg, wu, wd = (t[rank * el:(rank + 1) * el].contiguous() for t in synth.expert_weights(w, dev))
    s = r3.shape_of(wk)
    _, lg = r3.capture_topk_ws(s, 1, x, w_r, want_idx=False, want_logits=True)
    idx = synth.make_record(wk, lg)
    if args.ep_direct:
        # rows written straight into the owners' buffers (symmetric memory), outputs pulled by
        # address; capacity for the worst case (every row of every rank to one owner)
        state = EpDirectRank(rank, world, T, d, E, K, F)
        bufs = PeerBuffers.symmetric(world * T * K, d, wk.act_dtype, dev)

        def step():
            return ep_replay_layer_direct(state, bufs, x, w_r, idx, wg, wu, wd, dy)
    else:
        state = EpRank(rank, world, T, d, E, K, F)

        def step():
            return ep_replay_layer(state, x, w_r, idx, wg, wu, wd, dy)

    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    sampler = ClockSampler(local).start() if rank == 0 else None
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    dist.barrier()
    torch.cuda.synchronize()
    t0 = time.time()
    e0.record()
    for _ in range(args.steps):
        step()
    e1.record()
    torch.cuda.synchronize()
    dist.barrier()
    t1 = time.time()
    ms_total = r3dist.max_over_ranks(e0.elapsed_time(e1), dev)
    assert state.status.item() == 0
    if rank == 0:
        clocks = sampler.window(t0, t1)
        sampler.stop()
        ms = ms_total / args.steps
        line = {
            "metric": METRIC, "value": world * T / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": wk.name, "mode": (
                       "expert parallel, direct form: E/N experts and T tokens per rank, rows "
                       "written straight into the owners' symmetric-memory buffers, outputs pulled "
                       "by address, all-gather of the counts and three barriers per layer"
                       if args.ep_direct else
                       "expert parallel: E/N experts and T tokens per "
                       "rank, NCCL all-to-all of rows (torch.distributed) there and back"),
                       "T_per_gpu": T, "d": d, "E": E, "K": K, "F": F},
            "clocks": clocks, "peaks": peaks,
        }
        print(json.dumps(line), flush=True)
    dist.destroy_process_group()


def run_diag(args):
    """Discrepancy measures of Sections 3.1-3.2 (not the headline path): k3 KL + F(tau) over 10 M
    token probabilities (the paper's scatter sample), and the router/token-level comparison of two
    48-layer records of 65536 tokens.  One JSON line with achieved HBM GB/s per kernel."""
    import torch
    from paper_2510_11370_b200 import build
    build.build()
    from paper_2510_11370_b200 import r3
    if int(os.environ.get("RANK", "0")) != 0:
        return
    dev = torch.device("cuda", 0)
    peaks = load_peaks()
    g = torch.Generator(device=dev).manual_seed(0)
    n = 10_000_000
    pi = torch.rand(n, generator=g, device=dev) * 0.99 + 0.01
    pt = (pi * torch.exp(torch.randn(n, generator=g, device=dev) * 0.1)).clamp(1e-6, 1.0)
    taus = [1.05, 1.1, 1.5, 2.0, 4.0, 10.0]
    L, T, E, K = 48, 65536, 128, 8
    a = torch.argsort(torch.rand((L, T, E), generator=g, device=dev), dim=2)[:, :, :K].to(torch.uint8)
    b = a.clone()
    redo = torch.rand((L, T), generator=g, device=dev) < 0.1
    b[redo] = torch.argsort(torch.rand((int(redo.sum()), E), generator=g, device=dev), dim=1)[:, :K].to(torch.uint8)
    s = r3.make_shape(T, 8, E, K, 8)
    ws = r3.workspace(r3.lib.r3_prob_discrepancy_workspace_bytes(n), dev)

    def timed(fn, ring=1):
        """fn(i) runs the kernel on argument set i % ring."""
        for i in range(max(args.warmup, 3, ring)):
            fn(i % ring)
        torch.cuda.synchronize()
        return event_time(torch, lambda i: fn(i % ring), max(args.steps, 2 * ring))

    taus_d = torch.tensor(taus, dtype=torch.float32, device=dev)
    kl_o = torch.empty(1, dtype=torch.float64, device=dev)
    cnt_o = torch.empty(len(taus), dtype=torch.int64, device=dev)
    # inputs of 80 MB and 50 MB would stay in the 126 MB L2: each kernel walks a ring of copies
    n_p, n_r = ring_count(8 * n), ring_count(2 * L * T * K)
    pts, pis = [pt] + [pt.clone() for _ in range(n_p - 1)], [pi] + [pi.clone() for _ in range(n_p - 1)]
    ms_p = timed(lambda i: r3.prob_discrepancy(pts[i], pis[i], taus_d, kl=kl_o, counts=cnt_o, ws=ws),
                 n_p)
    del pts, pis
    ras, rbs = [a] + [a.clone() for _ in range(n_r - 1)], [b] + [b.clone() for _ in range(n_r - 1)]
    ms_r = timed(lambda i: r3.record_diff(s, L, ras[i], rbs[i], want_diff=False), n_r)
    del ras, rbs
    kl, counts = r3.prob_discrepancy(pt, pi, taus, ws=ws)
    # record store (Section 4.2): packed record of 4 sequences x 65536 tokens out of 16-token pages
    PT, Bq, Ts = 16, 4, 4 * 65536
    n_store_pages = Ts // PT
    page_bytes = r3.record_page_bytes(s, L, PT)
    pages = torch.randint(0, 128, (n_store_pages * page_bytes,), dtype=torch.uint8, device=dev)
    bt = torch.randperm(n_store_pages, generator=g, device=dev).to(torch.int32).reshape(Bq, -1).contiguous()
    cu = torch.arange(Bq + 1, dtype=torch.int32, device=dev) * (Ts // Bq)
    out_rec = torch.empty((L, Ts, K), dtype=torch.uint8, device=dev)
    ms_g = timed(lambda i: r3.record_gather(s, L, PT, pages, bt, cu, Ts, out=out_rec))
    pos0 = torch.zeros(Bq, dtype=torch.int32, device=dev)
    ms_a = timed(lambda i: r3.record_append(s, L, PT, pages, bt, pos0, cu, out_rec))
    # cpu_baseline leg: the oracle, as it stands, on a bounded sample
    from oracle import r3_diag_oracle as D
    t0 = time.perf_counter()
    m = 2_000_000
    ref_kl = D.kl_k3(pt[:m].cpu().numpy(), pi[:m].cpu().numpy())
    D.extreme_counts(pt[:m].cpu().numpy(), pi[:m].cpu().numpy(), taus)
    dt = time.perf_counter() - t0
    line = {
        "metric": "discrepancy-measure tokens/s (k3 KL + F(tau))", "value": n / (ms_p * 1e-3),
        "unit": "tokens/s", "n_gpus": 1, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_p, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f64", "data": "synthetic",
        "config": {"workload": "diag", "tokens": n, "taus": taus, "record": [L, T, K],
                   "l2": f"prob_discrepancy walks a ring of {n_p} input sets of 80 MB, record_diff "
                         f"one of {n_r} sets of 50 MB (more than twice the L2 in all); the record "
                         "store moves 200 MB per call"},
        "kernels": {
            "prob_discrepancy": {"ms": round(ms_p, 5), "hbm_gbs": round(8 * n / ms_p / 1e6, 1),
                                 "frac_of_measured_hbm": round(8 * n / ms_p / 1e6 / peaks["hbm_gbs"], 3)},
            "record_diff": {"ms": round(ms_r, 5),
                            "hbm_gbs": round(2 * L * T * K / ms_r / 1e6, 1),
                            "frac_of_measured_hbm": round(2 * L * T * K / ms_r / 1e6 / peaks["hbm_gbs"], 3)},
            "record_gather": {"ms": round(ms_g, 5), "hbm_gbs": round(2 * L * Ts * K / ms_g / 1e6, 1),
                              "frac_of_measured_hbm": round(2 * L * Ts * K / ms_g / 1e6 / peaks["hbm_gbs"], 3)},
            "record_append": {"ms": round(ms_a, 5), "hbm_gbs": round(2 * L * Ts * K / ms_a / 1e6, 1),
                              "frac_of_measured_hbm": round(2 * L * Ts * K / ms_a / 1e6 / peaks["hbm_gbs"], 3)}},
        "kl_k3": kl.item(), "F_tau": [c / n for c in counts.cpu().tolist()],
        "cpu_baseline": {"value": m / dt, "unit": "tokens/s", "cores": 1, "kind": "oracle",
                         "sample": f"first {m} tokens, kl_k3 + extreme_counts in numpy",
                         "kl_k3_of_sample": ref_kl},
        "peaks": peaks,
    }
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="all",
                    help="all (default: headline c4_replay plus every configuration under "
                         "per_config), one of the configurations, or diag")
    ap.add_argument("--ref-tokens", type=int, default=4096,
                    help="tokens of the workload the CPU oracle is timed on")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-sustained", action="store_true",
                    help="skip the regions of at least 0.6 s (for runs under a profiler)")
    ap.add_argument("--tokens", type=int, default=None,
                    help="with --workload: the same layer on this many tokens (profiling captures "
                         "on a case of a few GB); the line then names the workload 'name@T'")
    ap.add_argument("--stack", action="store_true", help="kept for old command lines: a multi-layer "
                    "workload is always timed over all its blocks")
    ap.add_argument("--ep", action="store_true",
                    help="expert-parallel layer: experts split over the ranks, all-to-all of rows")
    ap.add_argument("--ep-direct", action="store_true",
                    help="expert-parallel layer, rows written straight into the owners' buffers")
    ap.add_argument("--train", action="store_true",
                    help="time forward + the whole backward of one layer (bf16 workloads)")
    args = ap.parse_args()
    from paper_2510_11370_b200 import dist as r3dist, synth
    # `--gpus N` without a launcher: start the N ranks here (one process per GPU)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ and args.impl == "ours":
        sys.exit(r3dist.run_ranks(args.gpus, os.path.abspath(__file__), sys.argv[1:]))
    if args.workload == "diag":
        return run_diag(args)
    name = HEADLINE if args.workload == "all" else args.workload
    w = synth.WORKLOADS[name]
    if args.tokens:
        w = synth.WORKLOADS[name] = synth.scaled(w, name=f"{name}@{args.tokens}", T=args.tokens)
    if args.impl == "reference":
        return run_reference(args, w)
    if args.ep or args.ep_direct:
        return run_ep(args, synth.WORKLOADS["c2_layer_bf16"] if args.workload == "all" else w)
    if args.train and w.layers == 1:
        return run_train(args, synth.WORKLOADS["c2_layer_bf16"] if args.workload == "all" else w)
    run_ours(args)


if __name__ == "__main__":
    main()
