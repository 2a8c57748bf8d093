#!/usr/bin/env python
"""Benchmark of the MARS verification hot path (libmars) on B200.

One "step" is one full verification call over one batch: stream every logits row, top-2,
margin rule, longest accepted path, emit.  The default workload is the serving-scale
batched tree verification (256 sequences x 60-node depth-6 trees = 15 360 rows, |V| =
151 936, bf16 logits, 4.67 GB per step), the configuration on which the HBM-roofline target
is stated.  Prints ONE JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

With N > 1 (torchrun) every rank verifies its own batch of the same shape (sequences are
independent: no data-path collective); the time is the maximum over ranks.
`--impl reference` times the CPU oracle on the host cores instead of the CUDA library.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import sys
import threading
import time

import numpy as np
import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2601_15498_b200 import synth  # noqa: E402

METRIC = "verified_positions_per_sec"
UNIT = "positions/s"
L2_BYTES = 126 * 1024 * 1024
HBM_NOMINAL_GBS = 8000.0
HBM_FALLBACK_GBS = 6650.0

WORKLOADS = {
    "cfg3_bf16": lambda dev, seed, B=256: synth.cfg3(dev, seed=seed, B=B, dtype=torch.bfloat16),
    "cfg3_fp32": lambda dev, seed, B=256: synth.cfg3(dev, seed=seed, B=B, dtype=torch.float32),
    "cfg2": lambda dev, seed, B=64: synth.cfg2(dev, seed=seed, B=B),
    "cfg1": lambda dev, seed, B=1: synth.cfg1(dev, seed=seed, B=B),
    "cfg0": lambda dev, seed, B=1: synth.cfg0(dev, seed=seed, B=B),
}
FULL_NAME = {"cfg3_bf16": "cfg3_tree_b256_n60_v151936_bf16", "cfg3_fp32": "cfg3_tree_b256_n60_v151936_fp32",
             "cfg2": "cfg2_chain_b64_k8_v151936_bf16", "cfg1": "cfg1_tree_b1_n60_v151936_bf16",
             "cfg0": "cfg0_chain_b1_k6_v32000_fp32"}
BASE_SEED = {"cfg3_bf16": 3, "cfg3_fp32": 3, "cfg2": 2, "cfg1": 1, "cfg0": 0}


# ------------------------------------------------------------------------------ helpers

def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    except Exception:
        return HBM_FALLBACK_GBS, "fallback (earlier pool measurement)"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML while a region runs."""

    BAD = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20}
    NOTED = {"sw_power_cap": 0x4}

    def __init__(self, device_index: int, period_s: float = 0.02):
        self.period = period_s
        self.samples, self.reasons = [], set()
        self.max_mhz = None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            try:
                uuid = str(torch.cuda.get_device_properties(device_index).uuid)
                if not uuid.startswith("GPU-"):
                    uuid = "GPU-" + uuid
                self._h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
            except Exception:
                vis = os.environ.get("CUDA_VISIBLE_DEVICES")
                idx = int(vis.split(",")[device_index]) if vis and vis.split(",")[0].isdigit() else device_index
                self._h = pynvml.nvmlDeviceGetHandleByIndex(idx)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None

    def _poll(self):
        nv = self._nv
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self._h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self._h))
                for name, bit in {**self.BAD, **self.NOTED}.items():
                    if mask & bit:
                        self.reasons.add(name)
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        if self._h is not None:
            self._thread = threading.Thread(target=self._poll, daemon=True)
            self._thread.start()
        return self

    def __exit__(self, *a):
        self._stop.set()
        if self._thread:
            self._thread.join()

    def summary(self) -> dict:
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


def ncu_traffic(workload: str):
    """DRAM bytes per launch of the dominant kernel from the committed ncu summary, or None."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic_per_launch.txt")) as f:
            for line in f:
                parts = line.split()
                if len(parts) >= 2 and parts[0] == workload:
                    return int(parts[1])
    except Exception:
        pass
    return None


def reduce_max_time_sum_units(elapsed_ms: float, units: float, world: int):
    """Whole-job figures from per-rank ones: slowest rank's time, all ranks' units."""
    if world == 1:
        return elapsed_ms, units
    import torch.distributed as dist
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    t = torch.tensor([elapsed_ms], dtype=torch.float64, device=dev)
    u = torch.tensor([units], dtype=torch.float64, device=dev)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    dist.all_reduce(u, op=dist.ReduceOp.SUM)
    return float(t.item()), float(u.item())


def exp_unit_roofline(w, ms_per_step: float, clocks: dict):
    """Second ceiling of the stochastic path: one 2^x per logit on the SMs' exponential units
    (16 results per clock per SM, 148 SMs) at the SM clock sampled during the timed region."""
    mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965
    peak = 148 * 16 * mhz * 1e6 / 1e9
    achieved = w.R * w.V / (ms_per_step * 1e-3) / 1e9
    return {"bound": "alu", "unit": "G exp/s", "achieved": achieved, "peak": peak, "frac": achieved / peak,
            "peak_source": f"148 SMs x 16 per clock x {mhz:g} MHz (median sampled SM clock)"}


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


# ------------------------------------------------------------------------------ arms

def run_oracle_sample(w, host_logits, seqs: int, temperature=None, uniform=None):
    from oracle import mars_oracle as orc
    n = seqs * w.N
    t0 = time.perf_counter()
    if temperature is None:
        orc.verify_tree(host_logits[:n], w.tok[:seqs], w.parent[:seqs], w.theta)
    else:
        orc.verify_tree_stochastic(host_logits[:n], w.tok[:seqs], w.parent[:seqs], uniform[:seqs], w.theta,
                                   temperature)
    return time.perf_counter() - t0, n, orc.threads()


def stochastic_tag(args) -> str:
    return f"_stochastic_T{args.stochastic:g}" if args.stochastic else ""


def reference_arm(args, rank: int):
    """The CPU oracle, as it stands, on the host cores; rank 0 only."""
    if rank != 0:
        return
    seed = BASE_SEED[args.workload]
    if args.workload in ("cfg0", "cfg1"):
        w = WORKLOADS[args.workload]("cpu", seed)
    else:   # bounded sample: 16 whole sequences of the same recipe per step
        maker, kw = {"cfg3_bf16": (synth.cfg3, dict(dtype=torch.bfloat16)),
                     "cfg3_fp32": (synth.cfg3, dict(dtype=torch.float32)),
                     "cfg2": (synth.cfg2, {})}[args.workload]
        w = maker("cpu", seed=seed, B=16, **kw)
    seqs = w.B
    host = synth.to_numpy_bits(w.logits)
    uni = synth.make_uniforms(w.B, w.N, seed) if args.stochastic else None
    for _ in range(args.warmup):
        run_oracle_sample(w, host, seqs, args.stochastic, uni)
    t = 0.0
    cores = 1
    for _ in range(args.steps):
        dt, n, cores = run_oracle_sample(w, host, seqs, args.stochastic, uni)
        t += dt
    value = seqs * w.N * args.steps / t
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": FULL_NAME[args.workload] + stochastic_tag(args),
                   "logits_dtype": "bf16" if w.logits.dtype == torch.bfloat16 else "f32", "B": w.B, "N": w.N, "V": w.V, "theta": w.theta,
                   "note": "CPU oracle; each step is a bounded sample (B sequences) of the workload"},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                         "sample": f"{seqs} sequences x {w.N} rows per step"},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def measured_bf16_peak(sustained: bool):
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    key = "bf16_tflops_sustained" if sustained else "bf16_tflops"
    try:
        with open(path) as f:
            return float(json.load(f)[key]), f"measured (MEASURED_PEAKS.json, {key})"
    except Exception:
        return (1400.0 if sustained else 1590.0), "fallback (earlier pool measurement)"


def lmhead_arm(args, rank: int, world: int, local: int):
    """Fused LM-head + tree verification: hidden [64 x 60, 4096] bf16, W_vocab [151 936, 4096]
    bf16 (a model weight: resident in HBM in both the device-timed and the end-to-end figure),
    logits never stored.  Bound: tensor pipe (2 M d V flop per step)."""
    from paper_2601_15498_b200 import build, mars
    steps = 30 if args.steps is None else args.steps
    warm = 3 if args.warmup is None else max(args.warmup, 3)
    B = args.batch or 64
    if args.impl == "reference":
        if rank != 0:
            return
        from oracle import mars_oracle as orc
        w = synth.cfg4_operands("cpu", seed=4, B=1)
        hb, wb = synth.to_numpy_bits(w.hidden), synth.to_numpy_bits(w.w_vocab)
        tok = np.full((1, w.N), -1, np.int32)
        t = 0.0
        n = max(1, min(steps, 2))
        for _ in range(n):
            t0 = time.perf_counter()
            orc.lmhead_verify_tree(hb, wb, None, tok, w.parent, w.theta)
            t += time.perf_counter() - t0
        value = w.N * n / t
        print(json.dumps({
            "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": n, "warmup": 0, "ms_per_step": 1e3 * t / n, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": "cfg4_lmhead_b64_n60_v151936_d4096", "B": 1, "N": w.N, "V": w.V,
                       "d": w.d, "note": "fp64 oracle; each step is one sequence (60 rows)"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": orc.usable_cores(), "kind": "oracle",
                             "sample": "1 sequence x 60 rows per step (numpy fp64 matmul + C rule)"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}), flush=True)
        return

    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    barrier(world)
    w = synth.cfg4_operands(dev, seed=4 + 1000 * rank, B=B)
    M = w.B * w.N
    # draft tokens aim at the leading ids of a device fp32 matmul (inputs only)
    lead = np.empty((M, 2), np.int64)
    for r0 in range(0, M, 480):
        zz = w.hidden[r0:r0 + 480].float() @ w.w_vocab.float().T
        lead[r0:r0 + 480] = torch.topk(zz, 2, dim=1).indices.cpu().numpy()
        del zz
    tok_h = synth.make_tokens(w.parent, lead, w.V, 4)
    tok = torch.as_tensor(tok_h, device=dev)
    parent = torch.as_tensor(w.parent, device=dev)
    ws = torch.empty(int(mars.lib().mars_lmhead_workspace_bytes(w.B, w.N, w.V, w.d)), dtype=torch.uint8, device=dev)
    out = mars.alloc_outputs(w.B, w.N, w.N - 1, dev)
    flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)

    def step(h=None):
        mars.lmhead_verify(w.hidden if h is None else h, w.w_vocab, None, tok, parent, w.theta,
                           workspace=ws, out=out)

    for _ in range(warm):
        step()
    torch.cuda.synchronize()
    evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(steps)]
    barrier(world)
    with ClockSampler(local) as clocks:
        if args.profiler_range:
            torch.cuda.profiler.start()
        for a, b in evs:
            flush.zero_()                      # L2 flush between timed steps (outside the events)
            a.record()
            step()
            b.record()
        torch.cuda.synchronize()
        if args.profiler_range:
            torch.cuda.profiler.stop()
    barrier(world)
    elapsed_ms = sum(a.elapsed_time(b) for a, b in evs)
    total_ms, total_units = reduce_max_time_sum_units(elapsed_ms, float(M * steps), world)

    e2e = None
    if args.e2e_steps > 0:
        h_hidden = torch.empty(w.hidden.shape, dtype=w.hidden.dtype, pin_memory=True).copy_(w.hidden)
        h_tok, h_par = torch.as_tensor(tok_h).pin_memory(), torch.as_tensor(w.parent).pin_memory()
        h_out = {k: torch.empty(out[k].shape, dtype=out[k].dtype, pin_memory=True)
                 for k in ("accept_len", "out_tokens", "out_len")}
        d_hidden = torch.empty_like(w.hidden)

        def e2e_step():
            d_hidden.copy_(h_hidden, non_blocking=True)
            tok.copy_(h_tok, non_blocking=True)
            parent.copy_(h_par, non_blocking=True)
            step(d_hidden)
            for k, h in h_out.items():
                h.copy_(out[k], non_blocking=True)
        e2e_step()
        torch.cuda.synchronize()
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        f1.record()
        torch.cuda.synchronize()
        e_ms, e_units = reduce_max_time_sum_units(f0.elapsed_time(f1), float(M * args.e2e_steps), world)
        e2e = {"value": e_units / (e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": h_hidden.numel() * 2 + h_tok.numel() * 4 + h_par.numel() * 4,
               "d2h_bytes_per_step": sum(h.numel() * h.element_size() for h in h_out.values()),
               "steps": args.e2e_steps, "note": "W_vocab is a model weight and stays resident"}
    if rank != 0:
        return
    status = out["seq_status"].cpu().numpy()
    flops = 2.0 * M * w.d * w.V
    ms = elapsed_ms / steps
    tfs = flops / (ms * 1e-3) / 1e12
    peak, src = measured_bf16_peak(sustained=False)
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import mars_oracle as orc
        hb = synth.to_numpy_bits(w.hidden[:w.N])
        wb = synth.to_numpy_bits(w.w_vocab)
        t0 = time.perf_counter()
        orc.lmhead_verify_tree(hb, wb, None, tok_h[:1], w.parent[:1], w.theta)
        dt = time.perf_counter() - t0
        cpu = {"value": w.N / dt, "unit": UNIT, "cores": orc.usable_cores(), "kind": "oracle",
               "sample": f"first sequence ({w.N} rows): numpy fp64 projection + C rule, {dt:.1f} s"}
    print(json.dumps({
        "metric": METRIC, "value": total_units / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": warm, "ms_per_step": total_ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "N": w.N, "V": w.V, "d": w.d, "theta": w.theta,
                   "l2": "L2 flushed (252 MB write) before every timed step",
                   "all_sequences_ok": bool((status == 0).all())},
        "us_per_step": 1e3 * total_ms / steps, "tflops": tfs,
        "clocks": clocks.summary(), "e2e": e2e, "gpu_launches": 2 * steps,
        "roofline": {"bound": "tensor", "achieved": tfs, "peak": peak, "unit": "TFLOP/s",
                     "frac": tfs / peak, "traffic": None, "peak_source": src,
                     "kernel": "mars::lmhead_top2_kernel_pair", "algorithmic_flops_per_launch": flops},
        "cpu_baseline": cpu}), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_bf16", choices=sorted(WORKLOADS) + ["cfg4"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--profiler-range", action="store_true",
                    help="cudaProfilerStart/Stop around the timed region (for ncu --profile-from-start off)")
    ap.add_argument("--graph", action="store_true",
                    help="replay the steps from a CUDA graph (device time of launch-bound workloads)")
    ap.add_argument("--stochastic", type=float, default=None, metavar="T",
                    help="time stochastic verification at temperature T (Eq. 1 on the running residual + "
                         "draw) instead of the deterministic rule")
    ap.add_argument("--batch", type=int, default=None,
                    help="override the number of sequences (smaller cases for profiler captures)")
    args = ap.parse_args()

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))

    if args.workload == "cfg4":
        lmhead_arm(args, rank, world, local)
        return
    if args.impl == "reference":
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        reference_arm(args, rank)
        return

    args.steps = 2000 if args.steps is None else args.steps
    args.warmup = 10 if args.warmup is None else max(args.warmup, 3)

    from paper_2601_15498_b200 import build, mars
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    barrier(world)
    mars.lib()

    # ---- inputs, resident in HBM; every rank gets its own batch of the same shape ----
    if args.batch:
        w = WORKLOADS[args.workload](dev, BASE_SEED[args.workload] + 1000 * rank, args.batch)
    else:
        w = WORKLOADS[args.workload](dev, BASE_SEED[args.workload] + 1000 * rank)
    dt_code = mars.BF16 if w.logits.dtype == torch.bfloat16 else mars.FP32
    copies = 1
    if w.logits_bytes < 3 * L2_BYTES:   # small workloads: rotate over copies so that no step finds
        copies = -(-3 * L2_BYTES // w.logits_bytes)   # its rows in L2
    logits = [w.logits] + [w.logits.clone() for _ in range(copies - 1)]
    tok = torch.as_tensor(w.tok, device=dev)
    parent = torch.as_tensor(w.parent, device=dev)
    draft = torch.as_tensor(w.draft, device=dev)
    ws = torch.empty(mars.workspace_bytes(w.B, w.N, w.V, dt_code), dtype=torch.uint8, device=dev)
    out = mars.alloc_outputs(w.B, w.N, w.N - 1, dev)

    ws.zero_()
    fl = mars.COUNTERS_ZERO     # the workspace starts zeroed and every call leaves its counters at zero
    T = args.stochastic
    if T:
        uni_h = synth.make_uniforms(w.B, w.N, BASE_SEED[args.workload] + 1000 * rank)
        uni = torch.as_tensor(uni_h, device=dev)
        ws_s = torch.zeros(int(mars.lib().mars_stochastic_workspace_bytes(w.B, w.N, w.V, dt_code)),
                           dtype=torch.uint8, device=dev)
        out = mars.alloc_stochastic_outputs(w.B, w.N, w.N - 1, dev)

    def step(i, lg=None):
        lg = logits[i % copies] if lg is None else lg
        if T and w.kind == "chain":
            mars.verify_chain_stochastic(lg, draft, uni, w.theta, T, workspace=ws_s, out=out)
        elif T:
            mars.verify_tree_stochastic(lg, tok, parent, uni, w.theta, T, workspace=ws_s, out=out)
        elif w.kind == "chain":
            mars.verify_chain(lg, draft, w.theta, flags=fl, workspace=ws, out=out)
        else:
            mars.verify_tree(lg, tok, parent, w.theta, flags=fl, workspace=ws, out=out)

    for i in range(args.warmup):
        step(i)
    torch.cuda.synchronize()

    graph = None
    if args.graph:      # one graph = one pass over the rotating input copies
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(copies):
                step(i)
        replays = max(1, -(-args.steps // copies))
        args.steps = replays * copies
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()

    # ---- timed region: K steps between two events on the launching stream ----
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier(world)
    torch.cuda.synchronize()
    with ClockSampler(local) as clocks:
        if args.profiler_range:
            torch.cuda.profiler.start()
        e0.record()
        if graph is not None:
            for _ in range(replays):
                graph.replay()
        else:
            for i in range(args.steps):
                step(i)
        e1.record()
        torch.cuda.synchronize()
        if args.profiler_range:
            torch.cuda.profiler.stop()
    barrier(world)
    elapsed_ms = e0.elapsed_time(e1)
    total_ms, total_units = reduce_max_time_sum_units(elapsed_ms, float(w.R * args.steps), world)
    value = total_units / (total_ms * 1e-3)
    ms_per_step = total_ms / args.steps

    # ---- spread of single steps: an event pair around every repetition (median, p10, p90) ----
    reps = int(min(100, max(20, 200.0 / max(ms_per_step, 1e-3))))
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(reps)]
    for i, (a, b) in enumerate(pairs):
        a.record()
        if graph is not None:
            graph.replay()
        else:
            step(i)
        b.record()
    torch.cuda.synchronize()
    per = sorted(a.elapsed_time(b) * 1e3 / (copies if graph is not None else 1) for a, b in pairs)
    step_us = {"median": per[len(per) // 2], "p10": per[len(per) // 10], "p90": per[(9 * len(per)) // 10],
               "reps": reps, "note": ("per step of one graph replay" if graph is not None else
                                      "one event pair per step, launch gaps included")}

    # ---- this GPU's read-only ceiling on the same bytes: the library's streaming probe ----
    read_gbs = None
    if w.logits.is_contiguous() and w.logits_bytes >= 3 * L2_BYTES:
        row_bytes = w.V * w.logits.element_size()
        for _ in range(3):
            mars.stream_read_probe(w.logits, row_bytes)
        r0, r1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        r0.record()
        for _ in range(20):
            mars.stream_read_probe(w.logits, row_bytes)
        r1.record()
        torch.cuda.synchronize()
        read_gbs = w.logits_bytes * 20 / (r0.elapsed_time(r1) * 1e-3) / 1e9

    # ---- end to end: host buffers in, results out, copies inside the timed region ----
    e2e = None
    h_logits = None
    if args.e2e_steps > 0:
        h_logits = torch.empty(w.logits.shape, dtype=w.logits.dtype, pin_memory=True)
        h_logits.copy_(w.logits)
        h_tok = torch.as_tensor(w.tok).pin_memory()
        h_par = torch.as_tensor(w.parent).pin_memory()
        h_uni = torch.as_tensor(uni_h).pin_memory() if T else None
        h_out = {k: torch.empty(out[k].shape, dtype=out[k].dtype, pin_memory=True)
                 for k in ("accept_len", "out_tokens", "out_len")}
        d_logits = torch.empty_like(w.logits)

        def e2e_step():
            d_logits.copy_(h_logits, non_blocking=True)
            tok.copy_(h_tok, non_blocking=True)
            parent.copy_(h_par, non_blocking=True)
            if T:
                uni.copy_(h_uni, non_blocking=True)
            if w.kind == "chain":
                draft.copy_(tok[:, 1:])
            step(0, d_logits)
            for k, h in h_out.items():
                h.copy_(out[k], non_blocking=True)

        e2e_step()
        torch.cuda.synchronize()
        barrier(world)
        f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        f0.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        f1.record()
        torch.cuda.synchronize()
        e2e_ms, e2e_units = reduce_max_time_sum_units(f0.elapsed_time(f1), float(w.R * args.e2e_steps), world)
        h2d = w.logits_bytes + h_tok.numel() * 4 + h_par.numel() * 4 + (h_uni.numel() * 4 if T else 0)
        d2h = sum(h.numel() * h.element_size() for h in h_out.values())
        e2e = {"value": e2e_units / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": args.e2e_steps}

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    # ---- roofline of the one kernel on the path (algorithmic bytes: every logit once) ----
    peak, peak_src = measured_hbm_peak()
    achieved = w.logits_bytes / (elapsed_ms / args.steps * 1e-3) / 1e9
    traffic = ncu_traffic(args.workload + ("_stochastic" if T else "")) if not args.batch else None

    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        host = synth.to_numpy_bits(h_logits if h_logits is not None else w.logits)
        seqs = w.B          # the oracle finishes the whole batch in well under a minute
        run_oracle_sample(w, host, min(seqs, 2), T, uni_h if T else None)
        dt, n, cores = run_oracle_sample(w, host, seqs, T, uni_h if T else None)
        cpu = {"value": n / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"all {seqs} sequences ({n} rows) of the same workload, one pass, {dt:.2f} s"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name + stochastic_tag(args), "kind": w.kind,
                   "logits_dtype": "bf16" if w.logits.dtype == torch.bfloat16 else "f32",
                   "arithmetic": ("fp32 softmax weights 2^(z*log2(e)/T - ref) summed online, Eq. 1 on the running "
                                  "residual, fp64 partial sums in the draw" if T else
                                  "fp32 comparisons and one fp32 division per row (bf16 widens exactly)"),
                   "B": w.B, "N": w.N, "V": w.V,
                   "theta": w.theta, "rows_per_step": w.R, "logits_bytes_per_step": w.logits_bytes,
                   "l2": ("inputs larger than L2" if copies == 1 else
                          f"rotating over {copies} input copies, {copies * w.logits_bytes} B > L2"),
                   "launch": "cuda graph replay" if graph is not None else "direct launches",
                   "workspace": ("uninitialised (records only)" if T else
                                 "zeroed once; MARS_COUNTERS_ZERO (counters reset by the kernel itself)"),
                   "parallelism": f"dp{world} (independent sequences, no collective)"},
        "us_per_step": 1e3 * ms_per_step, "step_us": step_us,
        "hbm_gbs": achieved, "frac_of_8TBps_nominal": achieved / HBM_NOMINAL_GBS,
        "read_only_ceiling_gbs": read_gbs,
        "frac_of_read_only_ceiling": (achieved / read_gbs) if read_gbs else None,
        "clocks": clocks.summary(),
        "e2e": e2e,
        "gpu_launches": args.steps * (2 if T else 1),
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                     "frac": achieved / peak, "traffic": traffic, "peak_source": peak_src,
                     "kernel": "mars::stoch_stream_kernel" if T else "mars::verify_kernel",
                     "algorithmic_bytes_per_launch": w.logits_bytes,
                     **({"note": "duration = the whole step (streaming kernel + per-sequence tail kernel); the "
                                 "streaming kernel's own share is in profiles/",
                         "exp_unit": exp_unit_roofline(w, elapsed_ms / args.steps, clocks.summary())} if T else {})},
        "cpu_baseline": cpu,
    }
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
