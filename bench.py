#!/usr/bin/env python
"""Benchmark of the MARS verification hot path (libmars) on B200.

One "step" is one full verification call over one batch: stream every logits row, top-2,
margin rule, longest accepted path, emit.  The headline workload is the serving-scale batched
tree verification (256 sequences x 60-node depth-6 trees = 15 360 rows, |V| = 151 936, bf16
logits, 4.67 GB per step), the configuration on which the HBM-roofline target is stated.
Prints ONE JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]
                    [--shard seq|vocab] [--stochastic T] [--no-extras]

The default invocation (one GPU, headline workload) also measures, in the same process and the
same JSON line (`workloads`), every other configuration of the method -- the single chain, the
single tree, the batched chains, the fp32 batch, the fused LM head, stochastic verification at
T = 1, the vocabulary-sharded form, exact top-k selection and the telemetry histograms -- each
with its own roofline, read-only probe, clock record and an in-run comparison with the CPU
oracle (`parity`).

With N > 1 (torchrun) and `--shard seq` every rank verifies its own batch of the same shape
(sequences are independent: no data-path collective); with `--shard vocab` every rank streams its
column range of the same batch and the ranks exchange 16-byte records (one all-gather).  The time
is the maximum over ranks.  `--impl reference` times the CPU oracle on the host cores instead of
the CUDA library.
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
TOPK_WORKLOADS = [f"topk_k{k}_{d}" for k in (2, 10, 32) for d in ("bf16", "fp32")]

# stochastic comparison policy (the derivation is in tests/stochastic_checks.py's header)
PROB_RTOL, DECISION_TOL, DRAW_TOL = 2e-5, 2e-5, 1e-5


# ------------------------------------------------------------------------------ helpers

def measured_peaks():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return json.load(f)
    except Exception:
        return {}


def measured_hbm_peak():
    p = measured_peaks()
    if "hbm_gbs" in p:
        return float(p["hbm_gbs"]), "measured (MEASURED_PEAKS.json, copy bandwidth)"
    return HBM_FALLBACK_GBS, "fallback (earlier pool measurement)"


def measured_bf16_peak(sustained: bool):
    key = "bf16_tflops_sustained" if sustained else "bf16_tflops"
    p = measured_peaks()
    if key in p:
        return float(p[key]), f"measured (MEASURED_PEAKS.json, {key})"
    return (1400.0 if sustained else 1590.0), "fallback (earlier pool measurement)"


_NVML = {}


def _nvml_handle(device_index: int):
    """Read-only NVML handle of a CUDA device (cached); None when NVML is not usable."""
    if device_index in _NVML:
        return _NVML[device_index]
    h = None
    try:
        import pynvml
        pynvml.nvmlInit()
        try:
            uuid = str(torch.cuda.get_device_properties(device_index).uuid)
            if not uuid.startswith("GPU-"):
                uuid = "GPU-" + uuid
            h = pynvml.nvmlDeviceGetHandleByUUID(uuid)
        except Exception:
            vis = os.environ.get("CUDA_VISIBLE_DEVICES")
            idx = int(vis.split(",")[device_index]) if vis and vis.split(",")[0].isdigit() else device_index
            h = pynvml.nvmlDeviceGetHandleByIndex(idx)
        h = (pynvml, h, int(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM)))
    except Exception:
        h = None
    _NVML[device_index] = h
    return h


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU through NVML (queries only) while a
    region runs, about once a millisecond."""

    BAD = {"hw_slowdown": 0x8, "hw_thermal_slowdown": 0x40, "sw_thermal_slowdown": 0x20}
    NOTED = {"sw_power_cap": 0x4}

    def __init__(self, device_index: int, period_s: float = 0.001):
        self.period = period_s
        self.samples, self.reasons = [], set()
        self._stop = threading.Event()
        self._thread = None
        self._h = _nvml_handle(device_index)
        self.max_mhz = self._h[2] if self._h else None

    def _poll(self):
        nv, h, _ = self._h
        while not self._stop.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(h, nv.NVML_CLOCK_SM)))
                mask = int(nv.nvmlDeviceGetCurrentClocksEventReasons(h))
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
                "sm_min_mhz": min(self.samples) if self.samples else None,
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


def barrier(world: int):
    if world > 1:
        import torch.distributed as dist
        dist.barrier()


def pct(sorted_vals, q):
    return sorted_vals[min(len(sorted_vals) - 1, int(q * len(sorted_vals)))]


def ev():
    return torch.cuda.Event(enable_timing=True)


def timed_region(step, steps: int, warmup: int, *, copies: int = 1, graph_steps: int = 0, world: int = 1,
                 device_index: int = 0, spread_reps: int | None = None, profiler_range: bool = False, pre=None):
    """Times `step(i)` (which enqueues one step on the current stream, on input copy i % copies).

    Region A: `steps` steps between two events on the launching stream (barrier and synchronise on
    both sides) -- the throughput figure.  Region B: an event pair around every repetition, for the
    spread of single steps.  `graph_steps` > 0 replays the steps from a CUDA graph that
    holds that many of them (rounded up to whole passes over the copies).  `pre()` runs before
    every step outside the event pairs (an L2 flush).  The clock sampler stays open over both
    regions."""
    for i in range(warmup):
        if pre:
            pre()
        step(i)
    torch.cuda.synchronize()
    graph, per_graph = None, 1
    if graph_steps > 0:
        per_graph = -(-graph_steps // copies) * copies
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=side):
            for i in range(per_graph):
                step(i)
        for _ in range(2):
            graph.replay()
        torch.cuda.synchronize()
        replays = max(1, -(-steps // per_graph))
        steps = replays * per_graph
    e0, e1 = ev(), ev()
    barrier(world)
    torch.cuda.synchronize()
    with ClockSampler(device_index) as clocks:
        if profiler_range:
            torch.cuda.profiler.start()
        if pre is None:
            e0.record()
            if graph is not None:
                for _ in range(replays):
                    graph.replay()
            else:
                for i in range(steps):
                    step(i)
            e1.record()
            torch.cuda.synchronize()
            region_ms = e0.elapsed_time(e1)
        else:       # a flush between steps: every step gets its own event pair
            pairs = [(ev(), ev()) for _ in range(steps)]
            for i, (a, b) in enumerate(pairs):
                pre()
                a.record()
                step(i)
                b.record()
            torch.cuda.synchronize()
            region_ms = sum(a.elapsed_time(b) for a, b in pairs)
        if profiler_range:
            torch.cuda.profiler.stop()
        barrier(world)
        ms_per_step = region_ms / steps
        # ---- region B: spread (with a flush between steps region A already has one pair per step) ----
        if pre is None:
            if spread_reps is None:
                spread_reps = int(min(100, max(20, 100.0 / max(ms_per_step * per_graph, 1e-3))))
            pairs = [(ev(), ev()) for _ in range(spread_reps)]
            for i, (a, b) in enumerate(pairs):
                a.record()
                if graph is not None:
                    graph.replay()
                else:
                    step(i)
                b.record()
            torch.cuda.synchronize()
            spread_ms = sum(a.elapsed_time(b) for a, b in pairs)
        else:
            spread_reps, spread_ms = len(pairs), 0.0
        per = sorted(a.elapsed_time(b) * 1e3 / per_graph for a, b in pairs)
    ck = clocks.summary()
    med = pct(per, 0.5)
    return {
        "steps": steps, "region_ms": region_ms, "ms_per_step": ms_per_step,
        "step_us": {"median": med, "p10": pct(per, 0.1), "p90": pct(per, 0.9), "reps": spread_reps,
                    "note": (f"per step of one graph replay of {per_graph} steps" if graph is not None else
                             "one event pair per step, launch gaps included")},
        "launch": (f"cuda graph replay, {per_graph} steps per graph" if graph is not None else "direct launches"),
        "clocks": ck,
        "cycles_per_step": (ms_per_step * 1e3 * ck["sm_mhz"]) if ck["sm_mhz"] else None,
        "sampled_ms": region_ms + spread_ms,
    }


def hbm_roofline(bytes_per_launch: int, ms_per_step: float, kernel: str, traffic=None, **extra) -> dict:
    peak, src = measured_hbm_peak()
    achieved = bytes_per_launch / (ms_per_step * 1e-3) / 1e9
    return {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
            "traffic": traffic, "peak_source": src, "kernel": kernel,
            "algorithmic_bytes_per_launch": bytes_per_launch,
            "frac_of_8TBps_nominal": achieved / HBM_NOMINAL_GBS, **extra}


def read_probe(buffers, chunk_bytes: int, mars) -> dict:
    """This GPU's read-only ceiling on the same bytes, in the same launch arrangement: the
    library's streaming probe over each input copy in rotation (graph replay when one pass is
    short, so that launch gaps do not count against it)."""
    word = torch.zeros((1,), dtype=torch.int32, device=buffers[0].device)
    nbytes = buffers[0].numel() * buffers[0].element_size()

    def probe(i):
        mars.stream_read_probe(buffers[i % len(buffers)], chunk_bytes, out=word)

    est_us = max(nbytes / 7e12 * 1e6, 3.0)
    use_graph = est_us < 200.0
    steps = int(min(400, max(20, 20000.0 / est_us)))
    r = timed_region(probe, steps, 3, copies=len(buffers), graph_steps=(max(24, len(buffers)) if use_graph else 0),
                     spread_reps=20)
    us = r["step_us"]["median"]
    return {"gbs": nbytes / (us * 1e-6) / 1e9, "us": us, "launch": r["launch"],
            "mean_gbs": nbytes / (r["ms_per_step"] * 1e-3) / 1e9}


def exp_unit_roofline(R: int, V: int, ms_per_step: float, clocks: dict):
    """Second ceiling of the stochastic path: one 2^x per logit on the SMs' exponential units
    (16 results per clock per SM, 148 SMs) at the SM clock sampled during the timed region."""
    mhz = clocks.get("sm_mhz") or clocks.get("sm_max_mhz") or 1965
    peak = 148 * 16 * mhz * 1e6 / 1e9
    achieved = R * V / (ms_per_step * 1e-3) / 1e9
    return {"bound": "alu", "unit": "G exp/s", "achieved": achieved, "peak": peak, "frac": achieved / peak,
            "peak_source": f"148 SMs x 16 per clock x {mhz:g} MHz (median sampled SM clock)"}


# ------------------------------------------------------------------------------ parity

def _eq(a, b):
    return np.array_equal(a, b)


def parity_deterministic(got: dict, ref: dict, B: int, keys) -> dict:
    """Bit-exact comparison of GPU outputs with the oracle's, sequence by sequence."""
    bad = 0
    for b in range(B):
        if not all(_eq(got[k][b], ref[k][b]) for k in keys):
            bad += 1
    return {"checked_sequences": B, "mismatches": bad, "tolerance": "bit-exact (ids, lengths, paths, statuses)"}


def parity_stochastic(got: dict, ref: dict, B: int) -> dict:
    """Walks decided by more than DECISION_TOL must be identical; with the same walk the drawn token
    must be the oracle's unless the oracle's own draw lay within DRAW_TOL of a CDF step; node
    probabilities within PROB_RTOL.  Everything inside a tolerance is counted."""
    bad = close = neighbour = 0
    keys = ("accept_len", "path_nodes", "out_len", "seq_status", "node_how")
    for b in range(B):
        a = int(ref["accept_len"][b])
        same = all(_eq(got[k][b], ref[k][b]) for k in keys) and _eq(got["out_tokens"][b, :a], ref["out_tokens"][b, :a])
        if not same:
            if ref["margin"][b, 0] < DECISION_TOL:
                close += 1
            else:
                bad += 1
            continue
        if got["out_tokens"][b, a] != ref["out_tokens"][b, a]:
            if ref["margin"][b, 1] < DRAW_TOL:
                neighbour += 1
            else:
                bad += 1
    ok = ref["seq_status"][:B] != 1
    prob_bad = int((~np.isclose(got["node_prob"][:B][ok], ref["node_prob"][:B][ok], rtol=PROB_RTOL, atol=1e-30)).sum())
    return {"checked_sequences": B, "mismatches": bad + prob_bad, "decisions_within_tolerance": close,
            "draws_within_tolerance": neighbour,
            "tolerance": f"rule decisions bit-exact; Eq. 1 decisions closer than {DECISION_TOL:g} of the row's mass and "
                         f"draws closer than {DRAW_TOL:g} to a CDF step may differ; probabilities rtol {PROB_RTOL:g}"}


# ------------------------------------------------------------------------------ the verification cases

class VerifyCase:
    """One verification workload resident in HBM, with rotating input copies when it is smaller
    than three times the L2 cache."""

    def __init__(self, key: str, dev, mars, seed: int, batch=None, T=None, prebuilt=None):
        self.key, self.dev, self.mars, self.T = key, dev, mars, T
        if prebuilt is not None:
            self.w = w = prebuilt
        else:
            self.w = w = WORKLOADS[key](dev, seed, batch) if batch else WORKLOADS[key](dev, seed)
        self.dt_code = mars.BF16 if w.logits.dtype == torch.bfloat16 else mars.FP32
        self.copies = 1
        if w.logits_bytes < 3 * L2_BYTES:       # at least 8 copies, and more than 3 x L2 in total
            self.copies = max(8, -(-3 * L2_BYTES // w.logits_bytes))
        self.logits = [w.logits] + [w.logits.clone() for _ in range(self.copies - 1)]
        self.tok = torch.as_tensor(w.tok, device=dev)
        self.parent = torch.as_tensor(w.parent, device=dev)
        self.draft = torch.as_tensor(w.draft, device=dev)
        self.ws = torch.zeros(mars.workspace_bytes(w.B, w.N, w.V, self.dt_code), dtype=torch.uint8, device=dev)
        # workspace zeroed once and every call leaves its counters at zero; the logits are resident
        # before any step starts, so a step may stream them while the previous one drains
        self.flags = mars.COUNTERS_ZERO | mars.LOGITS_READY
        if T:
            self.uni_h = synth.make_uniforms(w.B, w.N, seed)
            self.uni = torch.as_tensor(self.uni_h, device=dev)
            self.ws_s = torch.zeros(int(mars.lib().mars_stochastic_workspace_bytes(w.B, w.N, w.V, self.dt_code)),
                                    dtype=torch.uint8, device=dev)
            self.out = mars.alloc_stochastic_outputs(w.B, w.N, w.N - 1, dev, debug=True)
        else:
            self.out = mars.alloc_outputs(w.B, w.N, w.N - 1, dev)

    @property
    def name(self):
        return self.w.name + (f"_stochastic_T{self.T:g}" if self.T else "")

    @property
    def launches_per_step(self):
        return 2 if self.T else 1

    def step(self, i, lg=None):
        w, m = self.w, self.mars
        lg = self.logits[i % self.copies] if lg is None else lg
        if self.T and w.kind == "chain":
            m.verify_chain_stochastic(lg, self.draft, self.uni, w.theta, self.T, flags=m.LOGITS_READY,
                                      workspace=self.ws_s, out=self.out)
        elif self.T:
            m.verify_tree_stochastic(lg, self.tok, self.parent, self.uni, w.theta, self.T, flags=m.LOGITS_READY,
                                     workspace=self.ws_s, out=self.out)
        elif w.kind == "chain":
            m.verify_chain(lg, self.draft, w.theta, flags=self.flags, workspace=self.ws, out=self.out)
        else:
            m.verify_tree(lg, self.tok, self.parent, w.theta, flags=self.flags, workspace=self.ws, out=self.out)

    def host_rows(self, seqs: int):
        return synth.to_numpy_bits(self.w.logits[:seqs * self.w.N])

    def oracle(self, host, seqs: int):
        from oracle import mars_oracle as orc
        w = self.w
        if self.T:
            return orc.verify_tree_stochastic(host, w.tok[:seqs], w.parent[:seqs], self.uni_h[:seqs], w.theta, self.T)
        if w.kind == "chain":
            return orc.verify_chain(host, w.draft[:seqs], w.theta)
        return orc.verify_tree(host, w.tok[:seqs], w.parent[:seqs], w.theta)

    def parity(self, seqs: int, ref=None):
        """Outputs of the buffers the timed steps wrote (every input copy holds the same data)
        against the oracle on the first `seqs` sequences."""
        got = self.mars.to_host(self.out)
        if ref is None:
            ref = self.oracle(self.host_rows(seqs), seqs)
        if self.T:
            return parity_stochastic(got, ref, seqs)
        keys = ("accept_len", "out_tokens", "out_len") if self.w.kind == "chain" else \
            ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status")
        return parity_deterministic(got, ref, seqs, keys)

    def probe(self):
        return read_probe(self.logits, self.w.V * self.w.logits.element_size(), self.mars)

    def config(self, world: int, launch: str, shard="seq") -> dict:
        w, T = self.w, self.T
        return {"workload": self.name, "kind": w.kind,
                "logits_dtype": "bf16" if w.logits.dtype == torch.bfloat16 else "f32",
                "arithmetic": ("fp32 softmax weights 2^(z*log2(e)/T - ref) summed online, Eq. 1 on the running "
                               "residual, fp64 partial sums in the draw" if T else
                               "fp32 comparisons and one fp32 division per row (bf16 widens exactly)"),
                "B": w.B, "N": w.N, "V": w.V, "theta": w.theta, "rows_per_step": w.R,
                "logits_bytes_per_step": w.logits_bytes,
                "l2": ("inputs larger than L2" if self.copies == 1 else
                       f"rotating over {self.copies} input copies, {self.copies * w.logits_bytes} B > L2"),
                "launch": launch,
                "overlap": "MARS_LOGITS_READY: the logits are resident before the step, so a call streams its rows "
                           "while the previous call on the stream drains (programmatic dependent launch) and "
                           "waits for it before touching workspace or outputs",
                "workspace": ("uninitialised (records only)" if T else
                              "zeroed once; MARS_COUNTERS_ZERO (counters reset by the kernel itself)"),
                "parallelism": f"dp{world} (independent sequences, no collective)"}


def small_entry(key: str, dev, mars, local: int, *, T=None, budget_ms: float = 60.0, parity_seqs=None,
                prebuilt=None) -> dict:
    """One entry of the `workloads` list for a stored-logits configuration."""
    c = VerifyCase(key, dev, mars, BASE_SEED[key], T=T, prebuilt=prebuilt)
    w = c.w
    est_us = max(w.logits_bytes / 6.5e12 * 1e6, 6.0) * (1.3 if T else 1.0)
    launch_bound = est_us < 200.0
    steps = int(min(4000, max(10, budget_ms * 1e3 / est_us)))
    gsteps = max(24, c.copies) if launch_bound else 0
    r = timed_region(c.step, steps, 5, copies=c.copies, graph_steps=gsteps, device_index=local)
    serialized = None
    if launch_bound:        # the same steps in plain stream order: what one call costs without overlap
        mars.test_hook(mars.HOOK_NO_OVERLAP, 1)
        try:
            r2 = timed_region(c.step, max(steps // 2, 10), 3, copies=c.copies, graph_steps=gsteps, device_index=local,
                              spread_reps=20)
        finally:
            mars.test_hook(mars.HOOK_NO_OVERLAP, 0)
        serialized = {"us_per_step": r2["ms_per_step"] * 1e3, "step_us": r2["step_us"],
                      "gbs": w.logits_bytes / (r2["ms_per_step"] * 1e-3) / 1e9,
                      "note": "same graph with every kernel launched in plain stream order (test hook): a call "
                              "cannot start before the previous one has finished"}
    pr = c.probe()
    seqs = w.B if parity_seqs is None else min(parity_seqs, w.B)
    us = r["ms_per_step"] * 1e3
    kernel = "mars::stoch_stream_kernel" if T else "mars::verify_kernel"
    roof = hbm_roofline(w.logits_bytes, r["ms_per_step"], kernel,
                        traffic=ncu_traffic(key + ("_stochastic" if T else "")))
    if T:
        roof["note"] = "duration = the whole step (streaming kernel + per-sequence tail kernel)"
        roof["exp_unit"] = exp_unit_roofline(w.R, w.V, r["ms_per_step"], r["clocks"])
    entry = {"workload": c.name, "rows_per_step": w.R, "logits_bytes_per_step": w.logits_bytes,
             "us_per_step": us, "step_us": r["step_us"], "serialized": serialized, "steps": r["steps"],
             "timed_region_ms": r["region_ms"], "launch": r["launch"], "l2": c.config(1, "")["l2"],
             "positions_per_s": w.R / (us * 1e-6), "gpu_launches_per_step": c.launches_per_step,
             "roofline": roof, "read_only_probe": pr, "frac_of_read_only_probe": roof["achieved"] / pr["mean_gbs"],
             "clocks": r["clocks"], "cycles_per_step": r["cycles_per_step"],
             "parity": c.parity(seqs)}
    if seqs < w.B:
        entry["parity"]["sample"] = f"first {seqs} of {w.B} sequences"
    return entry


# ------------------------------------------------------------------------------ vocabulary-parallel form

class VocabShardCase:
    """The same batch on every rank, each rank holding a contiguous column range: streaming
    top-2 of the shard, one all-gather of 16-byte records, merge + verification on every rank."""

    def __init__(self, key: str, dev, mars, rank: int, world: int, batch=None, prebuilt=None):
        from paper_2601_15498_b200 import vocab_parallel
        self.mars, self.world, self.rank = mars, world, rank
        if prebuilt is not None:
            full = prebuilt
        else:
            full = WORKLOADS[key](dev, BASE_SEED[key], batch) if batch else WORKLOADS[key](dev, BASE_SEED[key])
        self.w = full
        lo, hi = vocab_parallel.shard_ranges(full.V, world)[rank]
        self.lo, self.hi = lo, hi
        self.full_logits = full.logits if world == 1 else None
        self.local = full.logits if world == 1 else full.logits[:, lo:hi].contiguous()
        if world > 1:
            full.logits = None          # only the shard stays resident
            torch.cuda.empty_cache()
        self.dt_code = mars.BF16 if self.local.dtype == torch.bfloat16 else mars.FP32
        self.local_bytes = self.local.numel() * self.local.element_size()
        self.tok = torch.as_tensor(full.tok, device=dev)
        self.parent = torch.as_tensor(full.parent, device=dev)
        self.ws = torch.zeros(mars.workspace_bytes(full.B, full.N, hi - lo, self.dt_code), dtype=torch.uint8, device=dev)
        self.rec = torch.empty((full.R, 4), dtype=torch.int32, device=dev)
        self.gathered = torch.empty((world, full.R, 4), dtype=torch.int32, device=dev)
        self.out = mars.alloc_outputs(full.B, full.N, full.N - 1, dev)

    def step(self, i=0):
        m, w = self.mars, self.w
        m.top2_shard(self.local, w.B, w.N, self.lo, V_local=self.hi - self.lo, flags=m.COUNTERS_ZERO | m.LOGITS_READY,
                     workspace=self.ws, records=self.rec)
        if self.world > 1:
            import torch.distributed as dist
            dist.all_gather_into_tensor(self.gathered.view(self.world * w.R, 4), self.rec)
            recs = self.gathered
        else:
            recs = self.rec.view(1, w.R, 4)
        m.verify_records(recs, self.tok, self.parent, w.theta, out=self.out)


def vocab_entry(dev, mars, local: int, unsharded_out: dict | None, ref: dict | None, prebuilt) -> dict:
    """`workloads` entry for the vocabulary-sharded form on one GPU (one shard = the whole row):
    the same bytes through mars_top2_shard + mars_verify_records."""
    c = VocabShardCase("cfg3_bf16", dev, mars, 0, 1, prebuilt=prebuilt)
    w = c.w
    r = timed_region(c.step, 60, 5, device_index=local)
    got = mars.to_host(c.out)
    keys = ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status")
    par = parity_deterministic(got, ref, w.B, keys) if ref is not None else None
    same = None
    if unsharded_out is not None:
        same = all(_eq(got[k], unsharded_out[k]) for k in keys)
    us = r["ms_per_step"] * 1e3
    return {"workload": w.name + "_vocab_shards1", "rows_per_step": w.R, "logits_bytes_per_step": c.local_bytes,
            "us_per_step": us, "step_us": r["step_us"], "steps": r["steps"], "timed_region_ms": r["region_ms"],
            "launch": r["launch"], "positions_per_s": w.R / (us * 1e-6), "gpu_launches_per_step": 2,
            "roofline": hbm_roofline(c.local_bytes, r["ms_per_step"], "mars::verify_kernel (shard records)"),
            "clocks": r["clocks"], "cycles_per_step": r["cycles_per_step"], "parity": par,
            "bit_identical_to_unsharded_call": same}


def vocab_arm(args, rank: int, world: int, local: int):
    """`--shard vocab`: strong scaling over the vocabulary -- the batch is fixed, rank g streams
    columns [lo_g, hi_g) of every row; per step one all-gather of 16 B x rows per rank."""
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
    steps = 300 if args.steps is None else args.steps
    warm = 10 if args.warmup is None else max(args.warmup, 3)
    c = VocabShardCase(args.workload, dev, mars, rank, world, args.batch)
    w = c.w
    r = timed_region(c.step, steps, warm, world=world, device_index=local, profiler_range=args.profiler_range)
    total_ms, _ = reduce_max_time_sum_units(r["region_ms"], 0.0, world)
    units = float(w.R * r["steps"])        # every rank works on the same positions: counted once
    got = mars.to_host(c.out)
    parity = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        from oracle import mars_oracle as orc
        ref = orc.verify_tree(synth.to_numpy_bits(c.full_logits), w.tok, w.parent, w.theta)
        parity = parity_deterministic(got, ref, w.B, ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status"))
    if world > 1:
        import torch.distributed as dist
        # all ranks must hold identical outputs
        h = torch.as_tensor(np.concatenate([got[k].reshape(-1) for k in ("accept_len", "out_tokens", "out_len")]),
                            device=dev).to(torch.int64)
        lo_, hi_ = h.clone(), h.clone()
        dist.all_reduce(lo_, op=dist.ReduceOp.MIN)
        dist.all_reduce(hi_, op=dist.ReduceOp.MAX)
        parity = {"ranks_agree": bool((lo_ == hi_).all().item())}
    if rank == 0:
        ms = total_ms / r["steps"]
        line = {"metric": METRIC, "value": units / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world,
                "steps": r["steps"], "warmup": warm, "ms_per_step": ms, "higher_is_better": True,
                "scaling": "strong", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
                "config": {"workload": w.name + f"_vocab_shards{world}", "B": w.B, "N": w.N, "V": w.V,
                           "theta": w.theta, "rows_per_step": w.R, "columns_per_rank": c.hi - c.lo,
                           "logits_bytes_per_rank_per_step": c.local_bytes,
                           "l2": "inputs larger than L2" if c.local_bytes > 3 * L2_BYTES else
                                 "shard smaller than 3 x L2: partly L2-resident between steps",
                           "exchange": f"one all-gather of {16 * w.R} B per rank per step (NCCL), none at 1 GPU",
                           "units": "positions of the one shared batch, counted once (total work fixed as N grows)",
                           "parallelism": f"tp{world} over the vocabulary"},
                "us_per_step": ms * 1e3, "step_us": r["step_us"], "timed_region_ms": total_ms,
                "clocks": r["clocks"], "cycles_per_step": r["cycles_per_step"],
                "gpu_launches": 2 * r["steps"], "e2e": None, "parity": parity,
                "roofline": hbm_roofline(c.local_bytes, ms, "mars::verify_kernel (shard records)",
                                         note="per rank: the shard's bytes over the whole step (stream + gather + merge)"),
                "cpu_baseline": None}
        print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ------------------------------------------------------------------------------ top-k and telemetry

def topk_case(name: str, dev, mars, local: int, steps=None, warm=5, parity_rows: int = 256, batch=None) -> dict:
    """Exact top-k with ids over 7 680 rows of 151 936 logits (the drafter-side selection for
    top-k tree expansion)."""
    _, ks, dts = name.split("_")
    k = int(ks[1:])
    dtype = torch.bfloat16 if dts == "bf16" else torch.float32
    w = synth.cfg3(dev, seed=5, B=batch or 128, dtype=dtype)
    rows = w.R
    code = mars.BF16 if dtype == torch.bfloat16 else mars.FP32
    ws = torch.empty(int(mars.lib().mars_topk_workspace_bytes(rows, w.V, code, k)), dtype=torch.uint8, device=dev)
    out = (torch.empty((rows, k), dtype=torch.float32, device=dev), torch.empty((rows, k), dtype=torch.int32, device=dev))

    def step(i):
        mars.topk_rows(w.logits, k, workspace=ws, out=out)

    est_ms = w.logits_bytes / 3e12 * 1e3
    steps = steps or int(max(10, 50.0 / est_ms))
    r = timed_region(step, steps, warm, device_index=local)
    pr = read_probe([w.logits], w.V * w.logits.element_size(), mars)
    from oracle import mars_oracle as orc
    pick = np.unique(np.concatenate([np.arange(min(parity_rows // 2, rows)),
                                     np.arange(max(0, rows - parity_rows // 2), rows)]))
    host = synth.to_numpy_bits(w.logits[torch.as_tensor(pick, device=dev)])
    val_o, id_o = orc.topk(host, k)
    torch.cuda.synchronize()
    val_g, id_g = out[0].cpu().numpy()[pick], out[1].cpu().numpy()[pick]
    bad = int(((id_g != id_o).any(axis=1) | (val_g.view(np.uint32) != val_o.view(np.uint32)).any(axis=1)).sum())
    us = r["ms_per_step"] * 1e3
    roof = hbm_roofline(w.logits_bytes, r["ms_per_step"], "mars::topk_slice_kernel",
                        traffic=ncu_traffic(name) if rows == 7680 else None)
    return {"workload": f"topk_k{k}_rows{rows}_v{w.V}_{dts}", "rows_per_step": rows, "k": k,
            "logits_bytes_per_step": w.logits_bytes, "us_per_step": us, "step_us": r["step_us"], "steps": r["steps"],
            "timed_region_ms": r["region_ms"], "launch": r["launch"], "l2": "inputs larger than L2",
            "rows_per_s": rows / (us * 1e-6), "gpu_launches_per_step": 1 if rows > 296 else 2,
            "roofline": roof, "read_only_probe": pr, "frac_of_read_only_probe": roof["achieved"] / pr["mean_gbs"],
            "clocks": r["clocks"], "cycles_per_step": r["cycles_per_step"],
            "parity": {"checked_rows": int(len(pick)), "mismatches": bad,
                       "tolerance": "bit-exact (values and ids, best first)",
                       "sample": f"first and last {parity_rows // 2} rows"}}


def telemetry_entry(dev, mars, local: int, top2_val_host: np.ndarray) -> dict:
    """Histograms of z1, z2/z1, p2/p1 over the batch's top-2 values (inputs: the oracle's top-2
    of the same logits, uploaded -- the library's own top-2 is compared with it elsewhere)."""
    from oracle import mars_oracle as orc
    nb = 64
    v = torch.as_tensor(np.ascontiguousarray(top2_val_host, np.float32), device=dev)
    out = (torch.empty((3, nb), dtype=torch.int32, device=dev), torch.empty((3,), dtype=torch.int32, device=dev))

    def step(i):
        mars.top2_histograms(v, 0.0, 32.0, nb, out=out)

    r = timed_region(step, 480, 5, graph_steps=24, device_index=local)
    torch.cuda.synchronize()
    h_o, o_o = orc.histograms(top2_val_host, 0.0, 32.0, nb)
    bad = int((out[0].cpu().numpy().view(np.uint32) != h_o).sum() + (out[1].cpu().numpy().view(np.uint32) != o_o).sum())
    us = r["ms_per_step"] * 1e3
    return {"workload": f"telemetry_histograms_rows{v.shape[0]}_bins{nb}", "rows_per_step": int(v.shape[0]),
            "bytes_per_step": int(v.numel() * 4), "us_per_step": us, "step_us": r["step_us"],
            "steps": r["steps"], "timed_region_ms": r["region_ms"],
            "launch": r["launch"], "gpu_launches_per_step": 1,
            "roofline": {"bound": "latency", "note": "123 KB in, 780 B out per call: the call is one kernel "
                         "launch; no bandwidth or ALU ceiling applies"},
            "clocks": r["clocks"], "cycles_per_step": r["cycles_per_step"],
            "parity": {"checked_bins": 3 * nb + 3, "mismatches": bad, "tolerance": "exact counts"}}


# ------------------------------------------------------------------------------ fused LM head

class LmHeadCase:
    def __init__(self, dev, mars, seed: int, B: int):
        self.mars = mars
        self.w = w = synth.cfg4_operands(dev, seed=seed, B=B)
        M = w.B * w.N
        # draft tokens aim at the leading ids of a device fp32 matmul (inputs only)
        lead = np.empty((M, 2), np.int64)
        for r0 in range(0, M, 480):
            zz = w.hidden[r0:r0 + 480].float() @ w.w_vocab.float().T
            lead[r0:r0 + 480] = torch.topk(zz, 2, dim=1).indices.cpu().numpy()
            del zz
        self.tok_h = synth.make_tokens(w.parent, lead, w.V, 4)
        self.tok = torch.as_tensor(self.tok_h, device=dev)
        self.parent = torch.as_tensor(w.parent, device=dev)
        self.ws = torch.empty(int(mars.lib().mars_lmhead_workspace_bytes(w.B, w.N, w.V, w.d)), dtype=torch.uint8,
                              device=dev)
        self.out = mars.alloc_outputs(w.B, w.N, w.N - 1, dev, debug=True)
        self.flush = torch.empty(2 * L2_BYTES, dtype=torch.uint8, device=dev)
        self.drain = torch.zeros(2 * L2_BYTES, dtype=torch.uint8, device=dev)
        self.word = torch.zeros((1,), dtype=torch.int32, device=dev)

    def flush_l2(self):
        """Write a buffer of twice the L2 size, then stream another one through the cache with the
        read-only probe: the written lines are evicted (and written back) before the timed step
        starts instead of during it, and the step finds none of its inputs in L2."""
        self.flush.zero_()
        self.mars.stream_read_probe(self.drain, 1 << 20, out=self.word)

    def step(self, i=0, h=None):
        w = self.w
        self.mars.lmhead_verify(w.hidden if h is None else h, w.w_vocab, None, self.tok, self.parent, w.theta,
                                workspace=self.ws, out=self.out)

    def parity(self, sample):
        """fp64 projection + fp64 rule on whole sample sequences.  Tolerance: the GPU's top-2 logits
        within 2e-4 relative + 1e-5 of the fp64 logits at the same ids; another id only for fp64 logits
        that close (a near tie); another decision only where the oracle's |r - theta| <= 2e-3 or a near
        tie sits in that sequence."""
        from oracle import mars_oracle as orc
        w = self.w
        got = self.mars.to_host(self.out)
        rows = np.concatenate([np.arange(b * w.N, (b + 1) * w.N) for b in sample])
        hb = synth.to_numpy_bits(w.hidden)[rows]
        wb = synth.to_numpy_bits(w.w_vocab)
        z = np.empty((len(rows), w.V))
        for v0 in range(0, w.V, 16384):
            z[:, v0:v0 + 16384] = orc.lmhead_logits(hb, wb[v0:v0 + 16384])
        theta = float(np.float32(w.theta))
        ref = orc.verify_tree(z, self.tok_h[sample], w.parent[sample], theta)
        ids_g, val_g = got["top2_id"][rows], got["top2_val"][rows]
        ids_o, val_o = ref["top2_id"], ref["top2_val"]
        R = np.arange(len(rows))
        bad = 0
        tie_rows = set()
        for k in (0, 1):
            zg = z[R, ids_g[:, k]]
            bad += int((~np.isclose(val_g[:, k], zg, rtol=2e-4, atol=1e-5)).sum())
            for r in np.flatnonzero(ids_g[:, k] != ids_o[:, k]):
                if abs(zg[r] - val_o[r, k]) <= 2e-4 * abs(val_o[r, k]) + 1e-5:
                    tie_rows.add(int(r))
                else:
                    bad += 1
        near = np.abs(val_o[:, 1] / val_o[:, 0] - theta) <= 2e-3
        tolerated = 0
        for j, b in enumerate(sample):
            same = all(_eq(got[k][b], ref[k][j]) for k in ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status"))
            if same:
                continue
            rr = range(j * w.N, (j + 1) * w.N)
            if any(near[r] or r in tie_rows for r in rr):
                tolerated += 1
            else:
                bad += 1
        return {"checked_sequences": len(sample), "mismatches": bad, "near_tie_rows": len(tie_rows),
                "decisions_within_tolerance": tolerated, "sample": f"sequences {list(sample)}",
                "tolerance": "top-2 logits rtol 2e-4 + 1e-5 vs the fp64 projection; ids may differ at near ties; "
                             "decisions may differ where |r - theta| <= 2e-3 or at a near tie"}


def lmhead_measure(c: LmHeadCase, steps: int, warm: int, world: int, local: int, profiler_range=False):
    return timed_region(c.step, steps, warm, world=world, device_index=local, pre=c.flush_l2,
                        profiler_range=profiler_range)


def lmhead_entry(dev, mars, local: int) -> dict:
    c = LmHeadCase(dev, mars, 4, 64)
    w = c.w
    r = lmhead_measure(c, 12, 3, 1, local)
    M = w.B * w.N
    flops = 2.0 * M * w.d * w.V
    tfs = flops / (r["ms_per_step"] * 1e-3) / 1e12
    peak, src = measured_bf16_peak(sustained=False)
    us = r["ms_per_step"] * 1e3
    return {"workload": w.name, "rows_per_step": M, "us_per_step": us, "steps": r["steps"],
            "timed_region_ms": r["region_ms"], "launch": r["launch"],
            "l2": "L2 flushed (252 MB written, then 252 MB read through it) before every timed step", "positions_per_s": M / (us * 1e-6),
            "gpu_launches_per_step": 2, "tflops": tfs,
            "roofline": {"bound": "tensor", "achieved": tfs, "peak": peak, "unit": "TFLOP/s", "frac": tfs / peak,
                         "traffic": ncu_traffic("cfg4") if w.B == 64 else None, "peak_source": src,
                         "kernel": "mars::lmhead_top2_kernel_pair",
                         "algorithmic_flops_per_launch": flops, "frac_of_2250_nominal": tfs / 2250.0},
            "clocks": r["clocks"], "cycles_per_step": r["cycles_per_step"],
            "parity": c.parity([0, 63])}


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
    c = LmHeadCase(dev, mars, 4 + 1000 * rank, B)
    w, out, tok, parent = c.w, c.out, c.tok, c.parent
    M = w.B * w.N
    r = lmhead_measure(c, steps, warm, world, local, args.profiler_range)
    elapsed_ms = r["region_ms"]
    total_ms, total_units = reduce_max_time_sum_units(elapsed_ms, float(M * steps), world)

    e2e = None
    if args.e2e_steps > 0:
        h_hidden = torch.empty(w.hidden.shape, dtype=w.hidden.dtype, pin_memory=True).copy_(w.hidden)
        h_tok, h_par = torch.as_tensor(c.tok_h).pin_memory(), torch.as_tensor(w.parent).pin_memory()
        h_out = {k: torch.empty(out[k].shape, dtype=out[k].dtype, pin_memory=True)
                 for k in ("accept_len", "out_tokens", "out_len")}
        d_hidden = torch.empty_like(w.hidden)

        def e2e_step():
            d_hidden.copy_(h_hidden, non_blocking=True)
            tok.copy_(h_tok, non_blocking=True)
            parent.copy_(h_par, non_blocking=True)
            c.step(0, d_hidden)
            for k, h in h_out.items():
                h.copy_(out[k], non_blocking=True)
        e2e_step()
        torch.cuda.synchronize()
        f0, f1 = ev(), ev()
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
    cpu = parity = None
    if world == 1 and not args.no_cpu_baseline:
        from oracle import mars_oracle as orc
        hb = synth.to_numpy_bits(w.hidden[:w.N])
        wb = synth.to_numpy_bits(w.w_vocab)
        t0 = time.perf_counter()
        orc.lmhead_verify_tree(hb, wb, None, c.tok_h[:1], w.parent[:1], w.theta)
        dt = time.perf_counter() - t0
        cpu = {"value": w.N / dt, "unit": UNIT, "cores": orc.usable_cores(), "kind": "oracle",
               "sample": f"first sequence ({w.N} rows): numpy fp64 projection + C rule, {dt:.1f} s"}
        parity = c.parity(sorted({0, w.B - 1}))
    print(json.dumps({
        "metric": METRIC, "value": total_units / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world,
        "steps": steps, "warmup": warm, "ms_per_step": total_ms / steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": w.name, "B": w.B, "N": w.N, "V": w.V, "d": w.d, "theta": w.theta,
                   "l2": "L2 flushed (252 MB written, then 252 MB read through it) before every timed step",
                   "all_sequences_ok": bool((status == 0).all())},
        "us_per_step": 1e3 * total_ms / steps, "tflops": tfs, "timed_region_ms": total_ms,
        "clocks": r["clocks"], "cycles_per_step": r["cycles_per_step"], "e2e": e2e, "gpu_launches": 2 * steps,
        "roofline": {"bound": "tensor", "achieved": tfs, "peak": peak, "unit": "TFLOP/s",
                     "frac": tfs / peak, "traffic": ncu_traffic("cfg4") if (w.B == 64 and world == 1) else None,
                     "peak_source": src,
                     "kernel": "mars::lmhead_top2_kernel_pair", "algorithmic_flops_per_launch": flops},
        "parity": parity, "cpu_baseline": cpu}), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


# ------------------------------------------------------------------------------ reference arm

def run_oracle_sample(w, host_logits, seqs: int, temperature=None, uniform=None):
    from oracle import mars_oracle as orc
    n = seqs * w.N
    t0 = time.perf_counter()
    if temperature is None:
        ref = orc.verify_tree(host_logits[:n], w.tok[:seqs], w.parent[:seqs], w.theta)
    else:
        ref = orc.verify_tree_stochastic(host_logits[:n], w.tok[:seqs], w.parent[:seqs], uniform[:seqs], w.theta,
                                         temperature)
    return time.perf_counter() - t0, n, orc.threads(), ref


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
        dt, n, cores, _ = run_oracle_sample(w, host, seqs, args.stochastic, uni)
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


# ------------------------------------------------------------------------------ main

def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=None)
    ap.add_argument("--warmup", type=int, default=None)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg3_bf16", choices=sorted(WORKLOADS) + ["cfg4", "telemetry"] + TOPK_WORKLOADS)
    ap.add_argument("--shard", default="seq", choices=["seq", "vocab"],
                    help="how N > 1 ranks share the work: independent sequences (no collective) or column "
                         "ranges of the vocabulary (one all-gather of 16-byte records per step)")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-extras", action="store_true",
                    help="skip the `workloads` list (the other configurations) of the default invocation")
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
        if args.workload.startswith("topk") or args.workload == "telemetry":
            args.workload = "cfg3_bf16"
        args.steps = 3 if args.steps is None else args.steps
        args.warmup = 1 if args.warmup is None else args.warmup
        reference_arm(args, rank)
        return
    if args.shard == "vocab":
        vocab_arm(args, rank, world, local)
        return

    from paper_2601_15498_b200 import build, mars
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if args.workload.startswith("topk"):
        if rank == 0:
            build.build()
            mars.lib()
            e = topk_case(args.workload, dev, mars, local, steps=args.steps, warm=max(args.warmup or 5, 3),
                          batch=args.batch)
            print(json.dumps(e), flush=True)
        return

    if args.workload == "telemetry":
        if rank == 0:
            build.build()
            mars.lib()
            from oracle import mars_oracle as orc
            w = synth.cfg3(dev, seed=3, B=args.batch or 256)
            top2_host, _ = orc.top2(synth.to_numpy_bits(w.logits))      # inputs of the call: the oracle's top-2
            del w
            print(json.dumps(telemetry_entry(dev, mars, local, top2_host)), flush=True)
        return

    default_run = (args.workload == "cfg3_bf16" and world == 1 and not args.batch and not args.stochastic
                   and not args.graph and not args.profiler_range)
    extras = default_run and not args.no_extras
    args.steps = 2000 if args.steps is None else args.steps
    args.warmup = 10 if args.warmup is None else max(args.warmup, 3)

    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)
    if rank == 0:
        build.build()
    barrier(world)
    mars.lib()

    # ---- inputs, resident in HBM; every rank gets its own batch of the same shape ----
    T = args.stochastic
    c = VerifyCase(args.workload, dev, mars, BASE_SEED[args.workload] + 1000 * rank, batch=args.batch, T=T)
    w = c.w

    # ---- timed region: K steps between two events on the launching stream ----
    r = timed_region(c.step, args.steps, args.warmup, copies=c.copies,
                     graph_steps=(max(24, c.copies) if args.graph else 0), world=world, device_index=local,
                     profiler_range=args.profiler_range)
    args.steps = r["steps"]
    elapsed_ms = r["region_ms"]
    total_ms, total_units = reduce_max_time_sum_units(elapsed_ms, float(w.R * args.steps), world)
    value = total_units / (total_ms * 1e-3)
    ms_per_step = total_ms / args.steps
    timed_out = mars.to_host(c.out)          # what the timed steps wrote
    config = c.config(world, r["launch"])

    # ---- this GPU's read-only ceiling on the same bytes: the library's streaming probe ----
    probe = c.probe() if w.logits.is_contiguous() else None

    # ---- end to end: host buffers in, results out, copies inside the timed region.  The
    # deterministic path goes through the library's host-buffer entry point (one C-ABI call does the
    # copies in, the kernel and the copies out); the stochastic path copies with torch around the
    # device-buffer call ----
    e2e = None
    h_logits = None
    if args.e2e_steps > 0:
        h_logits = torch.empty(w.logits.shape, dtype=w.logits.dtype, pin_memory=True)
        h_logits.copy_(w.logits)
        h_tok = torch.as_tensor(w.tok).pin_memory()
        h_par = torch.as_tensor(w.parent).pin_memory()
        h_uni = torch.as_tensor(c.uni_h).pin_memory() if T else None
        if T:
            h_out = {k: torch.empty(c.out[k].shape, dtype=c.out[k].dtype, pin_memory=True)
                     for k in ("accept_len", "out_tokens", "out_len")}
            d_logits = torch.empty_like(w.logits)

            def e2e_step():
                d_logits.copy_(h_logits, non_blocking=True)
                c.tok.copy_(h_tok, non_blocking=True)
                c.parent.copy_(h_par, non_blocking=True)
                c.uni.copy_(h_uni, non_blocking=True)
                if w.kind == "chain":
                    c.draft.copy_(c.tok[:, 1:])
                c.step(0, d_logits)
                for k, h in h_out.items():
                    h.copy_(c.out[k], non_blocking=True)
            api = "torch copies around mars_verify_*_stochastic"
        else:
            h_out = mars.alloc_host_outputs(w.B, w.N - 1)
            staging = torch.empty(int(mars.lib().mars_verify_tree_host_staging_bytes(
                w.B, w.N, w.V, c.dt_code, w.logits.shape[1], w.N - 1)), dtype=torch.uint8, device=dev)

            def e2e_step():
                mars.verify_tree_host(h_logits, h_tok, h_par, w.theta, staging, h_out, V=w.V)
            api = "mars_verify_tree_host (copies in, kernel, copies out in one C-ABI call; chains as linear trees)"

        e2e_step()
        torch.cuda.synchronize()
        if not T:        # the host-buffer call must give what the device-buffer call gave
            for k in ("accept_len", "out_len"):
                assert np.array_equal(h_out[k].numpy(), timed_out[k]), k
        barrier(world)
        f0, f1 = ev(), ev()
        f0.record()
        for _ in range(args.e2e_steps):
            e2e_step()
        f1.record()
        torch.cuda.synchronize()
        e2e_ms, e2e_units = reduce_max_time_sum_units(f0.elapsed_time(f1), float(w.R * args.e2e_steps), world)
        h2d = w.logits_bytes + h_tok.numel() * 4 + h_par.numel() * 4 + (h_uni.numel() * 4 if T else 0)
        d2h = sum(h.numel() * h.element_size() for h in h_out.values())
        e2e = {"value": e2e_units / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": h2d,
               "d2h_bytes_per_step": d2h, "steps": args.e2e_steps, "api": api}
        if T:
            del d_logits
        else:
            del staging

    if rank != 0:
        if world > 1:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    # ---- roofline of the one kernel on the path (algorithmic bytes: every logit once) ----
    traffic = ncu_traffic(args.workload + ("_stochastic" if T else "")) if not args.batch else None
    roof = hbm_roofline(w.logits_bytes, elapsed_ms / args.steps,
                        "mars::stoch_stream_kernel" if T else "mars::verify_kernel", traffic)
    del roof["frac_of_8TBps_nominal"]
    if T:
        roof["note"] = ("duration = the whole step (streaming kernel + per-sequence tail kernel); the "
                        "streaming kernel's own share is in profiles/")
        roof["exp_unit"] = exp_unit_roofline(w.R, w.V, elapsed_ms / args.steps, r["clocks"])
    achieved = roof["achieved"]

    # ---- CPU oracle on the same inputs: the reported baseline, and the parity verdict of the timed outputs ----
    cpu = parity_head = ref = None
    if world == 1 and not args.no_cpu_baseline:
        host = synth.to_numpy_bits(h_logits if h_logits is not None else w.logits)
        seqs = w.B          # the oracle finishes the whole batch in well under a minute
        run_oracle_sample(w, host, min(seqs, 2), T, c.uni_h if T else None)
        if w.kind == "chain":
            t0 = time.perf_counter()
            ref = c.oracle(host, seqs)
            dt, n = time.perf_counter() - t0, seqs * w.N
            from oracle import mars_oracle as orc
            cores = orc.threads()
        else:
            dt, n, cores, ref = run_oracle_sample(w, host, seqs, T, c.uni_h if T else None)
        cpu = {"value": n / dt, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"all {seqs} sequences ({n} rows) of the same workload, one pass, {dt:.2f} s"}
        if T:
            parity_head = parity_stochastic(timed_out, ref, seqs)
        else:
            keys = ("accept_len", "out_tokens", "out_len") if w.kind == "chain" else \
                ("accept_len", "out_tokens", "path_nodes", "out_len", "seq_status")
            parity_head = parity_deterministic(timed_out, ref, seqs, keys)
        del host
    h_logits = None

    # ---- every other configuration, same process, same line ----
    workloads = []
    if extras:
        t_ex = time.perf_counter()
        top2_host = ref["top2_val"] if ref is not None else None
        try:
            workloads.append(vocab_entry(dev, mars, local, timed_out, ref, w))
        except Exception as e:      # an entry that fails is reported, never dropped silently
            workloads.append({"workload": "cfg3_bf16_vocab_shards1", "error": repr(e)})
        del c                       # the headline's logits stay (w) for the stochastic entry below
        torch.cuda.empty_cache()

        def stochastic_then_release():
            try:
                return small_entry("cfg3_bf16", dev, mars, local, T=1.0, budget_ms=80.0, parity_seqs=64, prebuilt=w)
            finally:
                w.logits = None

        # the three small configurations first: they leave the GPU nearly idle for a moment, so the
        # large entries after them start from the same clocks as the headline did
        jobs = [("cfg0", lambda: small_entry("cfg0", dev, mars, local)),
                ("cfg1", lambda: small_entry("cfg1", dev, mars, local)),
                ("cfg2", lambda: small_entry("cfg2", dev, mars, local)),
                ("cfg3_bf16_stochastic_T1", stochastic_then_release),
                ("cfg3_fp32", lambda: small_entry("cfg3_fp32", dev, mars, local, parity_seqs=64)),
                ("cfg4", lambda: lmhead_entry(dev, mars, local)),
                ("topk_k10_bf16", lambda: topk_case("topk_k10_bf16", dev, mars, local)),
                ("topk_k10_fp32", lambda: topk_case("topk_k10_fp32", dev, mars, local)),
                ("topk_k2_bf16", lambda: topk_case("topk_k2_bf16", dev, mars, local)),
                ("topk_k32_bf16", lambda: topk_case("topk_k32_bf16", dev, mars, local))]
        if top2_host is not None:
            jobs.append(("telemetry", lambda: telemetry_entry(dev, mars, local, top2_host)))
        for name, job in jobs:
            try:
                workloads.append(job())
            except Exception as e:
                workloads.append({"workload": name, "error": repr(e)})
            torch.cuda.empty_cache()
        extras_s = time.perf_counter() - t_ex

    parity = None
    if parity_head is not None:
        parity = {"headline": parity_head,
                  "checked_sequences": parity_head["checked_sequences"], "mismatches": parity_head["mismatches"]}
        for e in workloads:
            p = e.get("parity")
            if p:
                parity["checked_sequences"] += p.get("checked_sequences", 0)
                parity["mismatches"] += p["mismatches"]
            if "error" in e:
                parity["mismatches"] += 1
        parity["note"] = ("GPU outputs of the timed buffers against the CPU oracle on the same inputs, in this run; "
                          "per workload under `workloads[i].parity` (rows / bins where the unit is not a sequence)")

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": "f32", "data": "synthetic",
        "config": config,
        "us_per_step": 1e3 * ms_per_step, "step_us": r["step_us"],
        "timed_region_ms": total_ms, "cycles_per_step": r["cycles_per_step"],
        "hbm_gbs": achieved, "frac_of_8TBps_nominal": achieved / HBM_NOMINAL_GBS,
        "read_only_ceiling_gbs": probe["mean_gbs"] if probe else None,
        "frac_of_read_only_ceiling": (achieved / probe["mean_gbs"]) if probe else None,
        "clocks": r["clocks"],
        "e2e": e2e,
        "gpu_launches": args.steps * (2 if T else 1),
        "sm_count": mars.device_check(),
        "roofline": roof,
        "cpu_baseline": cpu,
        "parity": parity,
    }
    if extras:
        line["workloads"] = workloads
        line["extras_wall_s"] = extras_s
    print(json.dumps(line), flush=True)
    if world > 1:
        import torch.distributed as dist
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
