#!/usr/bin/env python
"""Benchmark of the attention hot path (forward of every chunk pair, LSE merge, backward).

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One step = one pass of the whole path over one synthetic microbatch: hydra_attn_fwd,
hydra_lse_merge (when the workload is chunked) and hydra_attn_bwd (D-prep, dK/dV kernel, dQ kernel).
The metric is causal-pair TFLOP/s: fwd = 2 * sum_pairs * h * (192 + 128), bwd counted as 2.5 x fwd.
Prints ONE JSON line (rank 0). With N > 1 (launched by torch.distributed.run) every rank processes
its own microbatch of the same shape: weak scaling, no data-path collective.
`--impl reference` times the fp64 CPU oracle, as it stands, on a bounded sample of the same workload.
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

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import hydra_workloads as hw  # noqa: E402

METRIC = "attention fwd+bwd TFLOP/s (causal pairs)"
UNIT = "TFLOP/s"
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# algorithmic FLOPs per causal (i, j) pair and head of each tensor-core kernel
FLOPS_PER_PAIR = {"fwd": 2.0 * (192 + 128),                  # S = QK^T and O = PV
                  "bwd_dkv": 2.0 * (192 + 128 + 128 + 192),  # S, dP, dV, dK: each needed once
                  "bwd_dq": 2.0 * 192}                       # dQ = dS K (its S, dP are recomputation)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


# --------------------------------------------------------------------------------------------------
# clocks during the timed region (read-only NVML queries)
# --------------------------------------------------------------------------------------------------
class ClockSampler(threading.Thread):
    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown",
               0x4: "sw_power_cap"}

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._halt = threading.Event()
        self.ok = False
        try:
            import pynvml
            pynvml.nvmlInit()
            self.nv = pynvml
            self.dev = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.dev, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def run(self):
        while self.ok and not self._halt.is_set():
            try:
                self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.dev, self.nv.NVML_CLOCK_SM))
                bits = self.nv.nvmlDeviceGetCurrentClocksEventReasons(self.dev) \
                    if hasattr(self.nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                    else self.nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.dev)
                for bit, name in self.REASONS.items():
                    if bits & bit:
                        self.reasons.add(name)
            except Exception:
                break
            self._halt.wait(0.01)

    def stop(self):
        self._halt.set()
        self.join(timeout=2)
        med = statistics.median(self.samples) if self.samples else None
        return {"sm_mhz": med, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(self.samples)}


# --------------------------------------------------------------------------------------------------
# reference arm: the oracle on the host cores, bounded sample
# --------------------------------------------------------------------------------------------------
def _pick_sample(w, rate: float, budget_s: float):
    """Leading sequences (then more heads) of `w` worth about `budget_s` at `rate` pairs*heads per second."""
    lengths, pairs = [], 0
    for length in w.lengths:
        cost = length * (length + 1) // 2
        if lengths and (pairs + cost) / rate > budget_s:
            break
        if not lengths and cost / rate > budget_s:          # even the first sequence is too long
            length = max(64, int((2.0 * budget_s * rate) ** 0.5))
            cost = length * (length + 1) // 2
        lengths.append(length)
        pairs += cost
    heads = 1
    if len(lengths) == len(w.lengths):                       # the whole batch fits: add heads
        heads = int(max(1, min(w.n_heads, budget_s * rate // max(pairs, 1))))
    return hw.Workload(w.name + "_sample", lengths, heads, cp_r=w.cp_r)


def oracle_sample(w, budget_s: float):
    """A bounded sample of the workload (leading sequences, leading heads) whose fwd+bwd takes about
    `budget_s` on this host. The oracle's rate depends on the problem size (threads, caches), so the
    size is chosen in two steps: from a small probe, then from a timed run of that first choice."""
    import oracle
    probe = hw.Workload("probe", [768], 1)
    x = probe.tensors([0])
    t0 = time.perf_counter()
    out, lse = oracle.attn_fwd(x["q"], x["k"], x["v"], probe.cu(), True, probe.scale)
    oracle.attn_bwd(x["q"], x["k"], x["v"], x["do"], probe.cu(), True, probe.scale, out, lse)
    rate = probe.causal_pairs_total / max(time.perf_counter() - t0, 1e-6)      # pairs*head / s
    first = _pick_sample(w, rate, budget_s / 4)
    sec = oracle_step(first)
    if sec > budget_s / 8:
        rate = first.causal_pairs_total * first.n_heads / sec
    else:                                                    # too short to trust: assume it scales
        rate = max(rate, first.causal_pairs_total * first.n_heads / max(sec, 1e-6))
    return _pick_sample(w, rate, budget_s)


def sample_desc(sample, w) -> str:
    return (f"first {len(sample.lengths)} sequence(s) ({sample.total} tokens), {sample.n_heads} head(s) of "
            f"{w.name}, fwd+bwd")


def oracle_step(sample):
    import oracle
    x = sample.tensors(list(range(sample.n_heads)))
    cu = sample.cu()
    t0 = time.perf_counter()
    out, lse = oracle.attn_fwd(x["q"], x["k"], x["v"], cu, True, sample.scale)
    if sample.cp_r:
        pairs = oracle.causal_pairs(cu, sample.cp_r)
        d = oracle.bwd_prep(x["do"], out)
        oracle.attn_bwd_pairs(x["q"], x["k"], x["v"], x["do"], cu, pairs, True, sample.scale, lse, d)
    else:
        oracle.attn_bwd(x["q"], x["k"], x["v"], x["do"], cu, True, sample.scale, out, lse)
    return time.perf_counter() - t0


def run_reference(args, w):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    budget = min(15.0, 150.0 / max(args.steps + args.warmup, 1))
    sample = oracle_sample(w, budget)
    for _ in range(args.warmup):
        oracle_step(sample)
    times = [oracle_step(sample) for _ in range(args.steps)]
    total = sum(times)
    flops = 3.5 * sample.flops_fwd() * args.steps
    value = flops / total / 1e12
    desc = sample_desc(sample, w)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
            "data": "synthetic", "config": {"workload": w.name, "sample": desc},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.n_threads(), "kind": "oracle",
                             "sample": desc},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# --------------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------------
def device_inputs(w, torch, seed_shift: int):
    from paper_2609_34318_b200.runner import bits_to_tensor
    T, h = w.total, w.n_heads
    t = {}
    for n in ("q", "k", "v", "do"):
        d = hw.D_V if n in ("v", "do") else hw.D_QK
        t[n] = torch.empty((T, h, d), dtype=torch.bfloat16, device="cuda")
        for a in range(h):
            t[n][:, a, :] = bits_to_tensor(hw.tensor_bits(n, T, [a], seed=hw.SEED + seed_shift))[:, 0, :]
    return t


def max_over_ranks(value_ms: float, dist, device) -> float:
    """The slowest rank's time: what a multi-GPU number is computed from. Works with any backend
    (`device` is where the backend wants its tensors: "cuda" for nccl, "cpu" for gloo)."""
    import torch
    tt = torch.tensor([value_ms], device=device, dtype=torch.float64)
    dist.all_reduce(tt, op=dist.ReduceOp.MAX)
    return float(tt.item())


def whole_job_value(world: int, flops_per_rank_step: float, steps: int, max_ms: float) -> float:
    """Weak scaling: every rank processes its own microbatch; TFLOP/s of all ranks together."""
    return world * flops_per_rank_step * steps / (max_ms * 1e-3) / 1e12


def measure_secondary(args, name: str, steps: int, peaks, peak_kind):
    """The other configuration the target is quoted on (the 256K sequence cut for a ring of four), timed the
    same way on the same GPU right after the headline workload: a few steps of forward of the 36 chunk pairs,
    merge and (banded) backward. Its inputs are seeded N(0,1) bf16 drawn on the device (the numpy recipe of the
    parity tests takes minutes at this size; the timing does not depend on the values)."""
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep

    w = hw.workload(name)
    cu = w.cu()
    pairs, part_rows = (None, 0)
    if w.cp_r:
        pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, w.cp_r)
    torch.cuda.reset_peak_memory_stats()
    held0 = torch.cuda.memory_allocated()
    gen = torch.Generator(device="cuda")
    gen.manual_seed(hw.SEED)
    t = {n: torch.randn((w.total, w.n_heads, hw.D_V if n in ("v", "do") else hw.D_QK), generator=gen,
                        device="cuda", dtype=torch.float32).to(torch.bfloat16) for n in ("q", "k", "v", "do")}
    step = AttnStep(cu, w.n_heads, pairs, part_rows, True, float(w.scale))
    stream = torch.cuda.current_stream()

    def one_step():
        step.forward(t["q"], t["k"], t["v"])
        step.backward(t["q"], t["k"], t["v"], t["do"])

    warm = 3
    for _ in range(warm):
        one_step()
    status, detail = step.poll()
    if status != 0:
        raise RuntimeError(f"{name}: device status {status} at item {detail}")
    sampler = ClockSampler(torch.cuda.current_device())
    P.hydra_profile_enable(True)
    P.hydra_profile_collect()
    torch.cuda.synchronize()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(steps):
        one_step()
    e1.record(stream)
    torch.cuda.synchronize()
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    kernel_ms, kernel_n = P.hydra_profile_collect()
    P.hydra_profile_enable(False)
    status, detail = step.poll()
    if status != 0:
        raise RuntimeError(f"{name}: device status {status} at item {detail}")
    step.forward(t["q"], t["k"], t["v"])
    mhz_fwd = P.hydra_poll_clocks(step.workspace)[0]
    step.backward(t["q"], t["k"], t["v"], t["do"])
    _, mhz_dkv, mhz_dq = P.hydra_poll_clocks(step.workspace)
    clocks["in_kernel_mhz"] = {"fwd": round(mhz_fwd), "bwd_dkv": round(mhz_dkv), "bwd_dq": round(mhz_dq)}
    held = torch.cuda.max_memory_allocated() - held0
    value = 3.5 * w.flops_fwd() * steps / (total_ms * 1e-3) / 1e12
    dominant = max(kernel_ms, key=lambda k: kernel_ms[k])
    work = FLOPS_PER_PAIR[dominant] * w.causal_pairs_total * w.n_heads if dominant in FLOPS_PER_PAIR else 0.0
    # the steps are seconds long and follow each other without a pause: the power-capped (sustained) peak
    peak = peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"])
    achieved = work / (kernel_ms[dominant] / steps * 1e-3) / 1e12
    merge_bytes = sum((int(n) + 1) * 260.0 * r * w.n_heads for n, r in merge_groups(pairs))
    merge_ms = kernel_ms.get("merge", 0.0) / steps
    out = {"workload": name, "value": value, "unit": UNIT, "steps": steps, "warmup": warm,
           "ms_per_step": total_ms / steps,
           "kernel_ms_per_step": {k: v / steps for k, v in kernel_ms.items()},
           "frac_of_bf16_peak": {"measured_burst": value / peaks["bf16_tflops"], "measured_sustained": value / peak},
           "roofline": {"kernel": dominant, "bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                        "peak_kind": f"{peak_kind} sustained bf16", "frac": achieved / peak,
                        "launches_per_step": kernel_n[dominant] / steps},
           "merge_gbs": merge_bytes / (merge_ms * 1e-3) / 1e9 if merge_ms > 0 else None,
           "bwd_bands": int(round(kernel_n.get("bwd_dkv", 0) / steps)), "band_scratch_gb": args.band_scratch_gb,
           "device_bytes_held": int(held), "clocks": clocks,
           "config": {"tokens": w.total, "heads": w.n_heads, "pairs": 0 if pairs is None else int(len(pairs)),
                      "causal_pairs": w.causal_pairs_total, "note": w.note,
                      "inputs": "seeded N(0,1) bf16 drawn on the device",
                      "l2": "inputs larger than L2 (no flush between iterations)"}}
    del step, t
    torch.cuda.empty_cache()
    return out


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    cu = w.cu()
    pairs, part_rows = (None, 0)
    if w.cp_r:
        pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, w.cp_r)
    t = device_inputs(w, torch, rank)
    # problems whose dS hand-off buffer is over the 4 GiB limit run their backward in bands of query rows
    P.hydra_set_bwd_band_scratch(int(args.band_scratch_gb * 2 ** 30))
    step = AttnStep(cu, w.n_heads, pairs, part_rows, True, float(w.scale))
    stream = torch.cuda.current_stream()

    def one_step():
        step.forward(t["q"], t["k"], t["v"])
        step.backward(t["q"], t["k"], t["v"], t["do"])

    for _ in range(max(args.warmup, 3)):
        one_step()
    status, detail = step.poll()
    if status != 0:
        raise RuntimeError(f"device status {status} at item {detail}")

    # ---- timed region: K steps, CUDA events on the launching stream, per-kernel events inside ----
    sampler = ClockSampler(local)
    P.hydra_profile_enable(True)
    P.hydra_profile_collect()
    launches0 = P.hydra_launch_count()
    barrier()
    sampler.start()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record(stream)
    for _ in range(args.steps):
        one_step()
    e1.record(stream)
    barrier()
    clocks = sampler.stop()
    total_ms = e0.elapsed_time(e1)
    launches = P.hydra_launch_count() - launches0
    kernel_ms, kernel_n = P.hydra_profile_collect()
    P.hydra_profile_enable(False)
    if world > 1:
        total_ms = max_over_ranks(total_ms, dist, "cuda")
    status, detail = step.poll()
    if status != 0:
        raise RuntimeError(f"device status {status} at item {detail}")
    # The clock inside the kernels, right after the timed region (same thermal and power state): the
    # driver's clock query above is sampled between kernels and reads the maximum even when a
    # power-capped kernel runs well below it.
    for _ in range(2):
        step.forward(t["q"], t["k"], t["v"])
        mhz_fwd = P.hydra_poll_clocks(step.workspace)[0]
        step.backward(t["q"], t["k"], t["v"], t["do"])
        _, mhz_dkv, mhz_dq = P.hydra_poll_clocks(step.workspace)
    clocks["in_kernel_mhz"] = {"fwd": round(mhz_fwd), "bwd_dkv": round(mhz_dkv), "bwd_dq": round(mhz_dq)}

    flops_step = 3.5 * w.flops_fwd()
    value = whole_job_value(world, flops_step, args.steps, total_ms)

    # ---- end to end through the C ABI with host buffers (pinned), copies inside the timed region ----
    e2e = None
    if not args.no_e2e:
        host = {n: v.cpu().pin_memory() for n, v in t.items()}
        T, h = w.total, w.n_heads
        ho = {"out": torch.empty((T, h, hw.D_V), dtype=torch.bfloat16).pin_memory(),
              "lse": torch.empty((h, T), dtype=torch.float32).pin_memory(),
              "dq": torch.empty((T, h, hw.D_QK), dtype=torch.bfloat16).pin_memory(),
              "dk": torch.empty((T, h, hw.D_QK), dtype=torch.bfloat16).pin_memory(),
              "dv": torch.empty((T, h, hw.D_V), dtype=torch.bfloat16).pin_memory()}
        del step
        torch.cuda.empty_cache()
        arena = torch.empty(P.hydra_host_step_arena_bytes(cu, h, pairs) + 256, dtype=torch.uint8, device="cuda")
        off = (-arena.data_ptr()) % 256
        arena_ptr, arena_bytes = arena.data_ptr() + off, arena.numel() - off

        def host_step():
            P.hydra_attn_fwd_bwd_host(host["q"], host["k"], host["v"], host["do"], cu, h, pairs, True,
                                      float(w.scale), ho["out"], ho["lse"], ho["dq"], ho["dk"], ho["dv"],
                                      arena_ptr, arena_bytes)

        e_steps = max(1, min(args.steps, 5))
        host_step()
        barrier()
        e0.record(stream)
        for _ in range(e_steps):
            host_step()
        e1.record(stream)
        barrier()
        e2e_ms = e0.elapsed_time(e1)
        if world > 1:
            e2e_ms = max_over_ranks(e2e_ms, dist, "cuda")
        h2d = sum(v.numel() * v.element_size() for v in host.values())
        d2h = sum(v.numel() * v.element_size() for v in ho.values())
        e2e = {"value": whole_job_value(world, flops_step, e_steps, e2e_ms), "unit": UNIT,
               "h2d_bytes_per_step": h2d, "d2h_bytes_per_step": d2h, "steps": e_steps,
               "ms_per_step": e2e_ms / e_steps}
        assert torch.isfinite(ho["dq"].float()).all()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- roofline of the dominant kernel ----
    peaks, peak_kind = measured_peaks()
    dominant = max(kernel_ms, key=lambda k: kernel_ms[k])
    # all launches of the kernel in one step together process the workload (a banded backward launches
    # it once per band), so the rate is the step's work over the step's time in that kernel
    launches_per_step = max(kernel_n[dominant], 1) / args.steps
    per_launch_ms = kernel_ms[dominant] / args.steps
    if dominant in FLOPS_PER_PAIR:
        work = FLOPS_PER_PAIR[dominant] * w.causal_pairs_total * w.n_heads
        # the tensor cores have been busy without a pause since the first warm-up step: against the
        # sustained (power-capped) figure when that is more than two seconds, else against the burst figure
        sustained = total_ms / args.steps * (args.steps + max(args.warmup, 3)) > 2000.0
        peak = peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"]
        roof = {"kernel": dominant, "bound": "tensor", "achieved": work / (per_launch_ms * 1e-3) / 1e12,
                "peak": peak, "unit": "TFLOP/s",
                "peak_kind": f"{peak_kind} {'sustained' if sustained else 'burst'} bf16"}
    else:
        th = w.total * w.n_heads
        work = th * 516.0 if dominant == "bwd_prep" else 0.0
        if dominant == "merge":
            work = sum((int(n) + 1) * 260.0 * rows * w.n_heads for n, rows in merge_groups(pairs))
        roof = {"kernel": dominant, "bound": "hbm", "achieved": work / (per_launch_ms * 1e-3) / 1e9,
                "peak": peaks["hbm_gbs"], "unit": "GB/s", "peak_kind": f"{peak_kind} copy"}
    roof["frac"] = roof["achieved"] / roof["peak"]
    roof["traffic"], roof["traffic_source"] = recorded_traffic(dominant, w.name)
    roof["ms_per_launch"] = per_launch_ms / launches_per_step
    roof["launches_per_step"] = launches_per_step

    # ---- the second configuration of the target (N = 1 only): a few steps of the 256K ring workload ----
    secondary = None
    if world == 1 and args.secondary not in ("", "none") and args.secondary != w.name:
        if args.no_e2e:
            del step
        else:
            del arena
        t.clear()
        torch.cuda.empty_cache()
        secondary = measure_secondary(args, args.secondary, args.secondary_steps, peaks, peak_kind)

    # ---- CPU baseline: the oracle on a bounded sample, rank 0, N = 1 only ----
    cpu = None
    if world == 1 and not args.no_cpu:
        import oracle
        sample = oracle_sample(w, 12.0)
        sec = oracle_step(sample)
        cpu = {"value": 3.5 * sample.flops_fwd() / sec / 1e12, "unit": UNIT, "cores": oracle.n_threads(),
               "kind": "oracle", "seconds": sec,
               "sample": sample_desc(sample, w)}

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": w.name, "tokens": w.total, "heads": w.n_heads, "sequences": len(w.lengths),
                       "d_qk": hw.D_QK, "d_v": hw.D_V, "pairs": 0 if pairs is None else int(len(pairs)),
                       "causal_pairs": w.causal_pairs_total, "note": w.note,
                       "l2": "inputs larger than L2 (no flush between iterations)",
                       "bwd_bands": int(round(kernel_n.get("bwd_dkv", 0) / args.steps)),
                       "band_scratch_gb": args.band_scratch_gb},
            "frac_of_bf16_peak": value / world / peaks["bf16_tflops"],
            "kernel_ms_per_step": {k: v / args.steps for k, v in kernel_ms.items()},
            "roofline": roof, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": int(launches),
            "clocks": clocks, "secondary": secondary}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def run_report(args, w):
    """Per-kernel report of one workload (a JSON object on stdout, not the one-line bench contract):
    median and best of every kernel over the repetitions, with L2 flushed between repetitions so that
    the HBM-bound kernels are measured against HBM; fwd-only / bwd-only / total rates against the
    measured burst, measured sustained and nominal peaks; merge and D-prep GB/s; the time of the first
    call of the shape (plan build and upload) against a steady call; and, with --per-sequence, every
    sequence of the batch timed alone next to its share of sum(L^2), the paper's load model."""
    import statistics
    import torch
    import paper_2609_34318_b200 as P
    from paper_2609_34318_b200.runner import AttnStep

    torch.cuda.set_device(0)
    cu = w.cu()
    pairs, part_rows = (None, 0)
    if w.cp_r:
        pairs, part_rows, _, _ = P.hydra_zigzag_pairs(cu, w.cp_r)
    t = device_inputs(w, torch, 0)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    stream = torch.cuda.current_stream()

    def timed_step(step, x):
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        step.forward(x["q"], x["k"], x["v"])
        step.backward(x["q"], x["k"], x["v"], x["do"])
        e1.record(stream)
        torch.cuda.synchronize()
        return e0.elapsed_time(e1)

    P.hydra_set_bwd_band_scratch(int(args.band_scratch_gb * 2 ** 30))
    t0 = time.perf_counter()
    step = AttnStep(cu, w.n_heads, pairs, part_rows, True, float(w.scale))
    first_ms = timed_step(step, t)
    first_wall_ms = 1e3 * (time.perf_counter() - t0)
    for _ in range(max(args.warmup, 3)):
        timed_step(step, t)
    P.hydra_profile_enable(True)
    P.hydra_profile_collect()
    rows = {k: [] for k in ("fwd", "merge", "bwd_prep", "bwd_dkv", "bwd_dq", "grad_cast", "step")}
    bands = 1
    for _ in range(args.steps):
        flush.zero_()                                        # 256 MB > L2: the next kernels start cold
        ms = timed_step(step, t)
        kernel_ms, kernel_n = P.hydra_profile_collect()
        bands = max(bands, int(kernel_n.get("bwd_dkv", 1)))
        for k in rows:
            rows[k].append(ms if k == "step" else kernel_ms.get(k, 0.0))
    P.hydra_profile_enable(False)
    peaks, peak_kind = measured_peaks()
    med = {k: statistics.median(v) for k, v in rows.items()}
    best = {k: min(v) for k, v in rows.items()}
    f_fwd = w.flops_fwd()
    kernels_ms = med["fwd"] + med["merge"] + med["bwd_prep"] + med["bwd_dkv"] + med["bwd_dq"] + med["grad_cast"]
    bwd_ms = med["bwd_prep"] + med["bwd_dkv"] + med["bwd_dq"] + med["grad_cast"]
    tf = lambda flops, ms: flops / (ms * 1e-3) / 1e12 if ms > 0 else None
    total = tf(3.5 * f_fwd, kernels_ms)
    th = w.total * w.n_heads
    merge_bytes = sum((int(n) + 1) * 260.0 * r * w.n_heads for n, r in merge_groups(pairs))
    gbs = lambda b, ms: b / (ms * 1e-3) / 1e9 if ms > 0 and b > 0 else None
    report = {
        "workload": w.name, "repetitions": args.steps, "l2": "256 MB written between repetitions",
        "median_ms": med, "best_ms": best,
        "tflops": {"total": total, "fwd_only": tf(f_fwd, med["fwd"] + med["merge"]), "bwd_only": tf(2.5 * f_fwd, bwd_ms),
                   "total_best": tf(3.5 * f_fwd, sum(best[k] for k in ("fwd", "merge", "bwd_prep", "bwd_dkv", "bwd_dq",
                                                                       "grad_cast")))},
        "bwd_bands": bands, "band_scratch_gb": args.band_scratch_gb,
        "of_peak": {"measured_burst": total / peaks["bf16_tflops"],
                    "measured_sustained": total / peaks.get("bf16_tflops_sustained", peaks["bf16_tflops"]),
                    "nominal_2250": total / 2250.0, "peaks": peak_kind},
        "merge_gbs": gbs(merge_bytes, med["merge"]), "bwd_prep_gbs": gbs(th * 516.0, med["bwd_prep"]),
        "hbm_peak_gbs": {"measured": peaks["hbm_gbs"], "nominal": 8000.0},
        "first_call_ms": {"device": first_ms, "wall_including_plan_build": first_wall_ms,
                          "steady_step_ms": med["step"],
                          "note": "first step of the process: module load, arena allocation, attribute set-up"},
    }
    # A NEW problem shape in a warm process (what every micro-batch of a training loop is): the same sequences in
    # reverse order, hence new cu_seqlens and new work tables, but the same work. Host-side table build, staging
    # and the asynchronous upload are inside the timed step; no allocation and no device-wide wait happen.
    rev = hw.Workload(w.name + "_reversed", list(reversed(w.lengths)), w.n_heads, cp_r=w.cp_r)
    cu_r = rev.cu()
    pairs_r, rows_r = (None, 0)
    if rev.cp_r:
        pairs_r, rows_r, _, _ = P.hydra_zigzag_pairs(cu_r, rev.cp_r)
    step_r = AttnStep(cu_r, rev.n_heads, pairs_r, rows_r, True, float(rev.scale))
    torch.cuda.synchronize()
    free_before = torch.cuda.mem_get_info()[0]
    t0 = time.perf_counter()
    new_shape_ms = timed_step(step_r, t)
    new_shape_wall_ms = 1e3 * (time.perf_counter() - t0)
    free_after = torch.cuda.mem_get_info()[0]
    again_ms = min(timed_step(step_r, t) for _ in range(3))
    report["plan_build_host_ms"] = {name: 1e3 * min(P.hydra_plan_build_seconds(kind, cu, w.n_heads, pairs) for _ in range(3))
                                    for name, kind in (("fwd", P.HYDRA_WS_FWD), ("merge", P.HYDRA_WS_MERGE),
                                                       ("bwd", P.HYDRA_WS_BWD))}
    report["new_shape_first_call_ms"] = {"device": new_shape_ms, "wall": new_shape_wall_ms, "same_shape_again": again_ms,
                                         "ratio_to_steady": new_shape_ms / again_ms,
                                         "device_memory_moved_bytes": int(free_before - free_after)}
    del step_r
    # The backward in its accumulating form (what a ring engine calls once per ring step) and the cast of
    # the fp32 accumulators to bf16: the pairs of the workload in one call (cost of the fp32
    # read-modify-write epilogues against the bf16 stores) and, for a cut workload, one call per ring step.
    acc = [torch.zeros((w.total, w.n_heads, d), dtype=torch.float32, device="cuda") for d in (hw.D_QK, hw.D_QK, hw.D_V)]
    grads = [torch.empty(a.shape, dtype=torch.bfloat16, device="cuda") for a in acc]
    all_pairs = pairs if pairs is not None else P.hydra_zigzag_pairs(cu, 0)[0]
    ring_step = P.hydra_zigzag_pairs(cu, w.cp_r)[3] if w.cp_r else None
    calls = [all_pairs] if ring_step is None else [all_pairs[ring_step == s_].copy() for s_ in range(int(ring_step.max()) + 1)]

    def accumulate_pass(call_list):
        for a in acc:
            a.zero_()
        flush.zero_()
        P.hydra_profile_collect()
        for sel in call_list:
            P.hydra_attn_bwd_accumulate(t["q"], t["k"], t["v"], step.out, step.lse, t["do"], cu, w.n_heads, sel, True,
                                        float(w.scale), acc[0], acc[1], acc[2], step.workspace)
        for a, g in zip(acc, grads):
            P.hydra_grad_cast(a, g)
        torch.cuda.synchronize()
        return P.hydra_profile_collect()[0]

    P.hydra_profile_enable(True)
    accumulate_pass([all_pairs])
    one_call = [accumulate_pass([all_pairs]) for _ in range(3)]
    by_step = [accumulate_pass(calls) for _ in range(3)] if len(calls) > 1 else None
    P.hydra_profile_enable(False)
    pick = lambda runs, k: statistics.median(r[k] for r in runs)
    cast_bytes = sum(a.numel() for a in acc) * 6.0
    report["accumulating_backward"] = {
        "one_call_ms": {k: pick(one_call, k) for k in ("bwd_prep", "bwd_dkv", "bwd_dq", "grad_cast")},
        "grad_cast_gbs": gbs(cast_bytes, pick(one_call, "grad_cast")),
        "grad_cast_bytes": cast_bytes,
    }
    if by_step:
        report["accumulating_backward"]["ring_steps"] = len(calls)
        report["accumulating_backward"]["by_step_ms"] = {k: pick(by_step, k) for k in ("bwd_prep", "bwd_dkv", "bwd_dq", "grad_cast")}
    # The local permutations around the head <-> sequence all-to-all of an inner Ulysses group of 4 (q of
    # this workload; 4 bytes moved per element), with L2 flushed before each.
    del acc, grads
    if w.n_heads % 4 == 0:
        send = torch.empty((4, w.total, w.n_heads // 4, hw.D_QK), dtype=torch.bfloat16, device="cuda")
        back = torch.empty_like(t["q"])
        P.hydra_profile_enable(True)
        runs = []
        for _ in range(5):
            flush.zero_()
            P.hydra_profile_collect()
            P.hydra_ulysses_pack(t["q"], w.total, w.n_heads, hw.D_QK, 4, send)
            torch.cuda.synchronize()
            pack_ms = P.hydra_profile_collect()[0]["ulysses"]
            flush.zero_()
            P.hydra_ulysses_unpack(send, w.total, w.n_heads, hw.D_QK, 4, back)
            torch.cuda.synchronize()
            runs.append((pack_ms, P.hydra_profile_collect()[0]["ulysses"]))
        P.hydra_profile_enable(False)
        assert torch.equal(back, t["q"])
        moved = t["q"].numel() * 4.0
        report["ulysses_cp4"] = {"bytes": moved, "pack_ms": statistics.median(r[0] for r in runs),
                                 "unpack_ms": statistics.median(r[1] for r in runs),
                                 "pack_gbs": gbs(moved, statistics.median(r[0] for r in runs)),
                                 "unpack_gbs": gbs(moved, statistics.median(r[1] for r in runs))}
        del send, back
    # Grouped-query form (eight query heads per KV head, as in the GQA model of Section 6): forward and the
    # accumulating backward, same q / dO, K and V of h / 8 heads.
    if w.n_heads % 8 == 0:
        h_kv = w.n_heads // 8
        kg, vg = t["k"][:, :h_kv].contiguous(), t["v"][:, :h_kv].contiguous()
        gacc = [torch.zeros((w.total, hh, d), dtype=torch.float32, device="cuda")
                for hh, d in ((w.n_heads, hw.D_QK), (h_kv, hw.D_QK), (h_kv, hw.D_V))]

        def gqa_pass():
            flush.zero_()
            P.hydra_profile_collect()
            P.hydra_attn_fwd_gqa(t["q"], kg, vg, cu, w.n_heads, h_kv, pairs, True, float(w.scale), step.out, step.lse,
                                 step.o_part if step.has_partials else None,
                                 step.lse_part if step.has_partials else None, part_rows, step.workspace)
            if step.has_partials:
                P.hydra_lse_merge(step.o_part, step.lse_part, part_rows, cu, w.n_heads, pairs, step.out, step.lse,
                                  step.workspace)
            P.hydra_attn_bwd_accumulate_gqa(t["q"], kg, vg, step.out, step.lse, t["do"], cu, w.n_heads, h_kv, pairs,
                                            True, float(w.scale), gacc[0], gacc[1], gacc[2], step.workspace)
            torch.cuda.synchronize()
            return P.hydra_profile_collect()[0]

        P.hydra_profile_enable(True)
        gqa_pass()
        gruns = [gqa_pass() for _ in range(3)]
        P.hydra_profile_enable(False)
        gms = {k: pick(gruns, k) for k in ("fwd", "merge", "bwd_prep", "bwd_dkv", "bwd_dq")}
        report["gqa_8_to_1"] = {"kv_heads": h_kv, "ms": gms, "tflops": tf(3.5 * f_fwd, sum(gms.values()))}
        del gacc, kg, vg
    # Heads of 128 / 128 with eight query heads per KV head (the shape of the paper's grouped-query model,
    # Section 6): same lengths, seeded N(0,1) inputs drawn on the device, forward and one-shot backward.
    if w.n_heads % 8 == 0:
        d, h_kv = 128, w.n_heads // 8
        gen = torch.Generator(device="cuda")
        gen.manual_seed(hw.SEED + 128)
        mk = lambda heads: torch.randn((w.total, heads, d), generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
        q8, k8, v8, do8 = mk(w.n_heads), mk(h_kv), mk(h_kv), mk(w.n_heads)
        out8 = torch.empty((w.total, w.n_heads, d), dtype=torch.bfloat16, device="cuda")
        dq8, dk8, dv8 = torch.empty_like(q8), torch.empty_like(k8), torch.empty_like(v8)
        ws8 = torch.empty(max(P.hydra_workspace_bytes_dims(k_, cu, w.n_heads, h_kv, d, d, pairs)
                              for k_ in (P.HYDRA_WS_FWD, P.HYDRA_WS_MERGE, P.HYDRA_WS_BWD)), dtype=torch.uint8, device="cuda")
        scale8 = float(np.float32(1.0 / np.sqrt(np.float32(d))))

        def d128_pass():
            flush.zero_()
            P.hydra_profile_collect()
            P.hydra_attn_fwd_dims(q8, k8, v8, cu, w.n_heads, h_kv, d, d, pairs, True, scale8, out8, step.lse,
                                  step.o_part if step.has_partials else None,
                                  step.lse_part if step.has_partials else None, part_rows, ws8)
            if step.has_partials:
                P.hydra_lse_merge(step.o_part, step.lse_part, part_rows, cu, w.n_heads, pairs, out8, step.lse, ws8)
            P.hydra_attn_bwd_dims(q8, k8, v8, out8, step.lse, do8, cu, w.n_heads, h_kv, d, d, pairs, True, scale8,
                                  dq8, dk8, dv8, ws8)
            torch.cuda.synchronize()
            return P.hydra_profile_collect()[0]

        P.hydra_profile_enable(True)
        d128_pass()
        druns = [d128_pass() for _ in range(3)]
        P.hydra_profile_enable(False)
        dms = {k: pick(druns, k) for k in ("fwd", "merge", "bwd_prep", "bwd_dkv", "bwd_dq", "grad_cast")}
        flops128 = 3.5 * 2.0 * w.causal_pairs_total * w.n_heads * (d + d)
        report["d128_gqa_8_to_1"] = {"kv_heads": h_kv, "ms": dms, "tflops": tf(flops128, sum(dms.values())),
                                     "flop_convention": "2 * pairs * h * (128 + 128) forward, backward 2.5 x"}
        del q8, k8, v8, do8, out8, dq8, dk8, dv8, ws8
    # The elementwise steps of a gated MLA block around the kernel (Section 5.2.2) on this workload's tokens and
    # heads: RoPE on the rotary slice of q (out of place), assembly of k / v from the up-projection and its
    # backward, the output gate and its backward; L2 flushed before each, rates over the algorithmic bytes.
    n, hh = w.total, w.n_heads
    d_nope, d_rope = hw.D_QK - 64, 64
    gen = torch.Generator(device="cuda")
    gen.manual_seed(hw.SEED + 7)
    rnd = lambda *shape: torch.randn(shape, generator=gen, device="cuda", dtype=torch.float32).to(torch.bfloat16)
    pos = (torch.arange(n, device="cuda", dtype=torch.int32) % 4096).contiguous()
    q_rot = torch.empty_like(t["q"])
    kv_up, k_pe = rnd(n, hh, d_nope + hw.D_V), rnd(n, d_rope)
    k_as, v_as = torch.empty_like(t["k"]), torch.empty_like(t["v"])
    dkv_up, dk_pe = torch.empty_like(kv_up), torch.empty_like(k_pe)
    gate, y = rnd(n, hh, hw.D_V), torch.empty_like(t["v"])
    d_out, d_gate = torch.empty_like(y), torch.empty_like(y)
    kv_bytes = (kv_up.numel() + k_pe.numel() + k_as.numel() + v_as.numel()) * 2.0
    ops = {
        "rope_q": (lambda: P.hydra_mla_rope(t["q"], pos, n, hh, hw.D_QK, d_nope, d_rope, 10000.0, False, q_rot),
                   t["q"].numel() * 4.0),
        "kv_assemble": (lambda: P.hydra_mla_kv_assemble(kv_up, k_pe, pos, n, hh, d_nope, d_rope, hw.D_V, 10000.0,
                                                        k_as, v_as), kv_bytes),
        "kv_assemble_bwd": (lambda: P.hydra_mla_kv_assemble_bwd(k_as, v_as, pos, n, hh, d_nope, d_rope, hw.D_V,
                                                                10000.0, dkv_up, dk_pe), kv_bytes),
        "gate": (lambda: P.hydra_gate_apply(t["v"], gate, y.numel(), y), y.numel() * 6.0),
        "gate_bwd": (lambda: P.hydra_gate_apply_bwd(y, t["v"], gate, y.numel(), d_out, d_gate), y.numel() * 10.0),
    }
    report["mla_elementwise"] = {}
    for name, (fn, nbytes) in ops.items():
        times = []
        for _ in range(5):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            fn()
            e1.record()
            torch.cuda.synchronize()
            times.append(e0.elapsed_time(e1))
        ms = statistics.median(times)
        report["mla_elementwise"][name] = {"ms": ms, "bytes": nbytes, "gbs": gbs(nbytes, ms)}
    del q_rot, kv_up, k_pe, k_as, v_as, dkv_up, dk_pe, gate, y, d_out, d_gate
    if args.per_sequence:
        # every sequence alone, same kernels: its share of the time next to its share of sum(L^2)
        shares = []
        for b, length in enumerate(w.lengths):
            lo = int(cu[b])
            xb = {n: v[lo:lo + length].contiguous() for n, v in t.items()}
            sb = AttnStep(hw.cu_seqlens([length]), w.n_heads, None, 0, True, float(w.scale))
            timed_step(sb, xb)
            shares.append((length, min(timed_step(sb, xb) for _ in range(3))))
        tsum = sum(ms for _, ms in shares)
        l2sum = float(sum(length * length for length, _ in shares))
        report["per_sequence"] = [{"L": length, "ms": ms, "time_share": ms / tsum, "L2_share": length * length / l2sum}
                                  for length, ms in sorted(shares, reverse=True)]
        report["per_sequence_note"] = ("short sequences sit above their share of sum(L^2): tile quantisation and the "
                                       "fixed cost of an item")
    print(json.dumps(report), flush=True)


def run_sched(args):
    """Scheduling time of the load-driven DCP scheduler (host only): the library's heap search on
    batches of the size the paper schedules (one global batch over a pool of G ranks), and the
    oracle's direct scans on a bounded sample of the same batch for context."""
    import math
    import paper_2609_34318_b200 as P
    from oracle import scheduler as S

    rng = np.random.default_rng(hw.SEED)
    out = []
    for G, tokens_per_rank in ((2048, 8192), (16384, 8192)):
        B = tokens_per_rank
        budget = G * B * 4                                   # four micro-batches' worth of tokens
        lengths, total = [], 0
        while total < budget:                                # long-tailed mix up to 256K (Section 2.2)
            L = int(min(262144, max(64, round(math.exp(rng.normal(math.log(1024), 1.4))))))
            lengths.append(L)
            total += L
        t = P.hydra_sched_targets(lengths, G, B, 4, 1e-9)
        C = max(t.C_star, t.C_mem)
        best = None
        for _ in range(5):
            t0 = time.perf_counter()
            mb, rank0, cp, n_mb = P.hydra_sched_pack(lengths, G, B, C)
            dt = time.perf_counter() - t0
            best = dt if best is None else min(best, dt)
        sample = lengths[:1500]
        Cs = max(C, S.ceil2(max(sample) / B))
        t0 = time.perf_counter()
        S.pack(sample, G, B, min(G, Cs))
        oracle_s = time.perf_counter() - t0
        out.append({"G": G, "B": B, "documents": len(lengths), "tokens": total, "C": int(C), "M_star": int(t.M_star),
                    "micro_batches": int(n_mb), "library_ms": 1e3 * best, "documents_per_s": len(lengths) / best,
                    "oracle_direct_scan_s_on_1500_documents": oracle_s})
    print(json.dumps({"scheduler": out}), flush=True)


def merge_groups(pairs):
    """(number of partials, rows) of every merged q chunk."""
    if pairs is None:
        return []
    out, i = [], 0
    while i < len(pairs):
        j = i
        while j < len(pairs) and pairs[j]["group"] == pairs[i]["group"]:
            j += 1
        if pairs[i]["part_row"] >= 0:
            out.append((j - i, int(pairs[i]["q_len"])))
        i = j
    return out


# dram__bytes_read.sum + dram__bytes_write.sum per launch, from ncu captures of this kernel on this workload
# (summaries with the full commands are kept with the other profiler summaries). Each figure carries the
# hash of the kernel sources it was captured from: when a source has changed since, the figure is no longer
# printed (traffic = null) instead of being repeated for a kernel it does not describe.
_TENSOR_DEPS = ("sm100_ptx.cuh", "hydra_internal.h")
NCU_DRAM_BYTES_PER_LAUNCH = {
    # (kernel, workload): (bytes per launch, source files, their hash at capture time, capture date)
    ("fwd", "packed32k"): (693289000, ("fwd_kernel.cu",) + _TENSOR_DEPS, "05986dad8ea8", "2026-11-25"),
    # with the dS hand-off: 1.76 GB of the key-side kernel's writes and of the query-side kernel's reads are dS
    ("bwd_dkv", "packed32k"): (2831744000, ("bwd_kernels.cu",) + _TENSOR_DEPS, "1fb384b3f8f2", "2026-11-25"),
    ("bwd_dq", "packed32k"): (2068468000, ("bwd_kernels.cu",) + _TENSOR_DEPS, "1fb384b3f8f2", "2026-11-25"),
    ("merge", "short64k_split"): (789849000, ("aux_kernels.cu", "hydra_internal.h", "sm100_ptx.cuh"), "a9b796e47f1c", "2026-11-25"),
    ("bwd_prep", "short64k_split"): (1086315000, ("aux_kernels.cu", "hydra_internal.h", "sm100_ptx.cuh"), "a9b796e47f1c", "2026-11-25"),
}


def kernel_source_hash(files) -> str:
    """Hash of the code of the listed kernel sources: comments and white space do not count, so that rewording
    a comment does not disown a capture of the same code."""
    import hashlib
    import re
    h = hashlib.sha1()
    for name in files:
        with open(os.path.join(ROOT, "paper_2609_34318_b200", "csrc", name), "r") as f:
            text = f.read()
        text = re.sub(r"/\*.*?\*/", " ", text, flags=re.S)
        text = re.sub(r"//[^\n]*", " ", text)
        h.update(" ".join(text.split()).encode())
    return h.hexdigest()[:12]


def recorded_traffic(kernel: str, workload: str):
    """(DRAM bytes per launch, where the figure comes from) for this kernel and workload; (None, why) if it was
    not captured or the kernel's sources have changed since the capture."""
    rec = NCU_DRAM_BYTES_PER_LAUNCH.get((kernel, workload))
    if rec is None:
        return None, "no ncu capture of this kernel on this workload"
    nbytes, files, src_hash, date = rec
    now = kernel_source_hash(files)
    if now != src_hash:
        return None, f"stale: ncu capture of {date} was of sources {src_hash}, the kernel is now {now}"
    return nbytes, f"ncu capture of {date}, kernel sources {src_hash} (dram__bytes_read.sum + dram__bytes_write.sum, one launch)"


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="packed32k", choices=list(hw.WORKLOADS))
    ap.add_argument("--band-scratch-gb", type=float, default=48.0,
                    help="dS scratch of the banded backward (long sequences only); 0 switches the bands off")
    ap.add_argument("--secondary", default="ring256k",
                    help="second workload timed after the headline one at N = 1 ('none' = skip it)")
    ap.add_argument("--secondary-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--report", action="store_true", help="per-kernel report of the workload instead of the bench line")
    ap.add_argument("--per-sequence", action="store_true", help="with --report: time every sequence alone")
    ap.add_argument("--sched", action="store_true", help="time the host scheduler instead (no GPU needed)")
    args = ap.parse_args()
    if args.sched:
        run_sched(args)
        return
    w = hw.workload(args.workload)
    if args.impl == "reference":
        run_reference(args, w)
    elif args.report:
        run_report(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
