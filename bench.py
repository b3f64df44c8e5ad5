#!/usr/bin/env python
"""Benchmark of the NetMax round simulator.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl ours|reference]

A step is one round: every worker of the workload draws a peer, takes its noisy SGD step and
pulls from the peer's round-start replica, over all M x d elements.  The metric is replica
GB/s = 16 bytes x M x d x rounds / time (reads of x_i, x_peer and c_i plus the write of x_i',
4 bytes each).  One JSON line is printed by rank 0.

The library advances up to eight rounds per launch where all M rows of a column tile fit in
shared memory (one CTA's up to 36 workers; four rounds over a thread-block cluster's beyond); that launch
is bound by instruction issue, not by HBM,
and the line's `roofline` says so.  The same workload with one launch per round (the HBM-bound
kernel) is timed as well and reported under `one_launch_per_round`.

With --gpus N > 1 (launched under torch.distributed.run) the replicas are sharded by columns:
every rank holds d columns of an N*d-long problem (weak scaling), draws the same peers from
the shared seed and exchanges nothing per round.

--impl reference times the CPU oracle (the only reference implementation there is) on a
bounded column sample of the same workload, on the host cores.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_2009_05766_b200 import workloads  # noqa: E402

BYTES_PER_ELEMENT = 16          # x_i, x_peer, c_i read + x_i' written, fp32: the replica GB/s metric counts these
BYTES_PER_ELEMENT_BF16 = 8      # the same four accesses with bfloat16 storage
UNIQUE_FRACTION = 0.75          # x_peer is a row the same tile reads anyway (a cache hit by design): 12 of the 16
                                # bytes (6 of 8) have to cross the DRAM pins, and the HBM roofline is taken against those
FALLBACK_HBM_GBS = 6650.0
NOMINAL_HBM_GBS = 8000.0
KERNEL_SOURCES = ("netmax_kernels.cuh", "netmax_rng.cuh")
# Counters of one launch, from ncu captures of this file's own commands (see profiles/): DRAM bytes
# (dram__bytes_read.sum + dram__bytes_write.sum) per element of the launch and warp instructions
# (smsp__inst_executed.sum) per element and round.  Captured on the workload itself where that is small
# enough to profile, else on the same M and tile shape with a shorter vector (`captured_on`); bytes and
# instructions per element are what carries over.  Only reported while the kernel sources still hash to
# the value the capture was taken at.
NCU_HASH = "a822180d1ad9aa37"
NCU_COUNTERS = {
    # (workload tag, kernel): dram bytes per element-launch, warp instructions per element-round, captured on
    ("cfg2_M8_resnet18", "round_kernel"): (1_041_843_000 / 89_391_696, 78_504_733 / 89_391_696, "cfg2"),
    ("cfg2_M8_resnet18", "fused_rounds_kernel"): (1_041_110_000 / 89_391_696, 612_995_880 / (89_391_696 * 8), "cfg2"),
    ("cfg2_M8_resnet18/bf16", "round_kernel"): (507_135_000 / 89_391_696, 85_164_099 / 89_391_696, "cfg2"),
    ("cfg2_M8_resnet18/bf16", "fused_rounds_kernel"): (505_620_000 / 89_391_696, 660_744_326 / (89_391_696 * 8), "cfg2"),
    ("cfg3_M16_vgg19scale", "fused_rounds_kernel"): (3_805_327_000 / 320_000_000, 2_031_045_889 / (320_000_000 * 8), "cfg3"),
    ("cfg3_M16_vgg19scale", "round_kernel"): (1_543_966_000 / (16 * 8_000_002), 101_887_293 / (16 * 8_000_002), "cfg3 at d = 8,000,002"),
    ("cfg4_M64_resnet18", "cluster_rounds_kernel"): (1_503_694_000 / (64 * 2_000_002), 524_126_023 / (64 * 2_000_002 * 4), "cfg4 at d = 2,000,002"),
    ("cfg4_M64_resnet18", "round_kernel"): (1_545_154_000 / (64 * 2_000_002), 104_626_918 / (64 * 2_000_002), "cfg4 at d = 2,000,002"),
    ("cfg1_M4_d4096", "resident_rounds_kernel"): (None, 49_802_752 / (16_384 * 1024), "cfg1"),
    ("cfg5_M4096_sampling", "resident_rounds_kernel"): (None, 5_822_930_304 / (4_194_304 * 1024), "cfg5"),
}
# Busy fractions (of active SM cycles) of the issue slots and of the arithmetic pipes, from the same captures on
# shorter vectors of the same M: which unit a launch that is bound by instruction issue leans on hardest.
NCU_PIPES = {
    ("cfg2_M8_resnet18", "fused_rounds_kernel"): {"issue": 0.600, "fmaheavy": 0.657, "fmalite": 0.296, "alu": 0.370,
                                                   "captured_on": "cfg2 at d = 4,000,002"},
    ("cfg3_M16_vgg19scale", "fused_rounds_kernel"): {"issue": 0.557, "fmaheavy": 0.639, "fmalite": 0.292, "alu": 0.345,
                                                      "captured_on": "cfg3 at d = 8,000,002"},
    ("cfg4_M64_resnet18", "cluster_rounds_kernel"): {"issue": 0.486, "fmaheavy": 0.499, "fmalite": 0.197, "alu": 0.339,
                                                      "captured_on": "cfg4 at d = 2,000,002"},
}
SM_COUNT, SCHEDULERS_PER_SM = 148, 4     # one warp instruction per scheduler and clock at most


def hash_sources(paths) -> str:
    """Hash of the code in C++ sources: `//` comments (the kernel sources have no other kind, and no `//` inside a
    string) and blank lines do not count, so that a reworded comment does not void the counters."""
    h = hashlib.sha256()
    for path in paths:
        with open(path, "r", encoding="utf-8") as f:
            for line in f:
                code = line.split("//", 1)[0].rstrip()
                if code:
                    h.update(code.encode("utf-8") + b"\n")
    return h.hexdigest()[:16]


def kernel_source_hash() -> str:
    return hash_sources(os.path.join(ROOT, "paper_2009_05766_b200", "csrc", name) for name in KERNEL_SOURCES)


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons of one GPU while the timed region runs."""

    REASONS = {"hw_slowdown": 0x8, "sw_thermal_slowdown": 0x20, "hw_thermal_slowdown": 0x40,
               "hw_power_brake_slowdown": 0x80, "sw_power_cap": 0x4}

    def __init__(self, index: int, period_s: float = 0.02):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._nvml = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nvml = pynvml
            self._handle = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._handle, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._nvml = None

    def _once(self):
        if self._nvml is not None:
            n = self._nvml
            self.samples.append(int(n.nvmlDeviceGetClockInfo(self._handle, n.NVML_CLOCK_SM)))
            mask = int(n.nvmlDeviceGetCurrentClocksThrottleReasons(self._handle))
            for name, bit in self.REASONS.items():
                if mask & bit:
                    self.reasons.add(name)
        else:
            out = subprocess.run(
                ["nvidia-smi", f"--id={self.index}", "--format=csv,noheader,nounits",
                 "--query-gpu=clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,"
                 "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
                 "clocks_event_reasons.sw_power_cap"], capture_output=True, text=True, timeout=10).stdout
            f = [v.strip() for v in out.strip().split(",")]
            self.samples.append(int(float(f[0])))
            self.max_mhz = int(float(f[1]))
            for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[2:]):
                if v.lower().startswith("active"):
                    self.reasons.add(name)

    def _run(self):
        while not self._stop.is_set():
            try:
                self._once()
            except Exception:
                pass
            self._stop.wait(self.period)

    def __enter__(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        return self

    def __exit__(self, *exc):
        self._stop.set()
        self._thread.join(timeout=15)

    def summary(self):
        return {"sm_mhz": statistics.median(self.samples) if self.samples else None, "sm_max_mhz": self.max_mhz,
                "reasons": sorted(self.reasons), "samples": len(self.samples)}


# ---------------------------------------------------------------------------- CPU oracle legs
def oracle_policy_inputs(w):
    """P, rho and the link graph for the oracle legs, from the oracle's own Algorithm 3."""
    from oracle import policy as opolicy
    s = w.link_speeds(0)
    if w.M > 256:   # the plain numpy Algorithm 3 is too slow here; speed-proportional rows stand in
        P = s / s.sum(axis=1, keepdims=True)
        adj = (s > 0).astype(np.uint8)
        off = ~np.eye(w.M, dtype=bool)
        return P, float((1 - 1e-6) * (P[off] / (2.0 * w.lr)).min()), adj
    t, adj = opolicy.iteration_times(s, w.d)
    P, rho, _ = opolicy.generate_policy(t, adj, w.lr, min(w.K, 6), min(w.R, 6))
    return P, rho, adj


def time_oracle(w, n_cols: int, rounds: int, warm: int, threads: int, storage: str = "f32"):
    """Seconds per round of the oracle on the first n_cols columns of all M replicas."""
    from oracle import oracle
    P, rho, adj = oracle_policy_inputs(w)
    cols = np.arange(n_cols, dtype=np.int64)
    sim = oracle.Sim(w.M, w.d, P, adj, alpha=w.lr, rho=rho, sigma=w.sigma, objective=1, seed=w.seed, cols=cols,
                     storage=storage)
    sim.init(w.x0_std, w.c_std)
    sim.round(warm, threads=threads)
    t0 = time.perf_counter()
    sim.round(rounds, threads=threads)
    dt = (time.perf_counter() - t0) / max(rounds, 1)
    sim.close()
    return dt


def cpu_baseline(w, budget_s: float = 15.0, storage: str = "f32"):
    threads = max(1, min(os.cpu_count() or 1, 64))
    bpe = BYTES_PER_ELEMENT_BF16 if storage == "bf16" else BYTES_PER_ELEMENT
    probe_cols = int(min(w.d, max(4096, 200_000 // w.M)))
    per_round = time_oracle(w, probe_cols, 2, 1, threads, storage)
    rate = w.M * probe_cols / per_round                       # elements per second
    rounds = 5
    n_cols = int(min(w.d, max(probe_cols, rate * budget_s / (rounds * w.M))))
    per_round = time_oracle(w, n_cols, rounds, 1, threads, storage)
    gbs = bpe * w.M * n_cols / per_round / 1e9
    one_cols = int(min(w.d, max(4096, rate / threads * 4.0 / (2 * w.M))))       # about 4 s on one thread
    one = time_oracle(w, one_cols, 2, 1, 1, storage)
    return {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle",
            "sample": f"first {n_cols} of {w.d} columns of all {w.M} replicas, {rounds} rounds, "
                      f"{threads} threads over column blocks",
            "rounds_per_s_extrapolated": n_cols / per_round / w.d,
            "value_1_thread": bpe * w.M * one_cols / one / 1e9}


def run_reference(args, w):
    """The oracle as the reference arm: K timed steps of a bounded column sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    threads = max(1, min(os.cpu_count() or 1, 64))
    probe_cols = int(min(w.d, max(4096, 200_000 // w.M)))
    bpe = BYTES_PER_ELEMENT_BF16 if args.storage == "bf16" else BYTES_PER_ELEMENT
    per_round = time_oracle(w, probe_cols, 2, 1, threads, args.storage)
    rate = w.M * probe_cols / per_round
    budget = 90.0
    n_cols = int(min(w.d, max(1024, rate * budget / ((args.steps + args.warmup) * w.M))))
    per_round = time_oracle(w, n_cols, args.steps, args.warmup, threads, args.storage)
    gbs = bpe * w.M * n_cols / per_round / 1e9
    sample = (f"first {n_cols} of {w.d} columns of all {w.M} replicas per step, {threads} threads")
    line = {
        "impl": "reference", "metric": "replica GB/s", "value": gbs, "unit": "GB/s", "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": per_round * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "d": w.d, "storage": args.storage, "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": "GB/s", "cores": threads, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": "GB/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------- GPU arm
def shard_plan(d: int, world: int, rank: int, align: int = 4):
    """Weak scaling by columns: rank g holds logical elements [g*d4, g*d4 + d) of a world*d4-long
    vector, d4 = d rounded up to a multiple of `align` (counter alignment: 4 elements per Philox
    block; 8 with bfloat16 storage, whose 16-byte column groups hold two blocks)."""
    d4 = (d + align - 1) // align * align
    return {"element_offset": rank * d4, "d": d, "global_d": world * d4}


def counters_for(tag: str, kernel: str):
    """(dram bytes per element-launch, warp instructions per element-round, captured_on) or Nones."""
    if kernel_source_hash() != NCU_HASH:
        return None, None, None
    return NCU_COUNTERS.get((tag, kernel), (None, None, None))


def hbm_roofline(tag, kernel, ms_per_round, elements, bpe, peak, peak_kind):
    """HBM-bound launch (one round per launch): achieved = the bytes that must cross the DRAM pins
    (12 of the 16 per element: the peer read is a cache hit by design) / time, against the measured
    copy peak; the DRAM bytes ncu counted for the same launch and the 16-byte metric ride along."""
    sec = ms_per_round / 1e3
    unique = UNIQUE_FRACTION * bpe * elements
    per_el, _, captured_on = counters_for(tag, kernel)
    traffic = None if per_el is None else per_el * elements
    out = {"bound": "hbm", "achieved": unique / sec / 1e9, "peak": peak, "unit": "GB/s",
           "frac": unique / sec / 1e9 / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}", "kernel": kernel,
           "bytes_per_launch": unique, "algorithmic_bytes_per_element": UNIQUE_FRACTION * bpe,
           "replica_GBs": bpe * elements / sec / 1e9}
    if traffic is not None:
        out.update({"dram_GBs": traffic / sec / 1e9, "dram_frac_of_measured": traffic / sec / 1e9 / peak,
                    "dram_frac_of_8TBs": traffic / sec / 1e9 / NOMINAL_HBM_GBS, "traffic_captured_on": captured_on})
    return out


def issue_roofline(tag, kernel, ms_per_round, elements, bpe, rounds_per_launch, sm_max_mhz, peak, peak_kind):
    """Launches that keep a tile on chip for several rounds are bound by instruction issue:
    achieved = warp instructions per second (ncu count per element and round x elements / time)
    against 148 SMs x 4 schedulers x 1 warp instruction per clock at clocks.max.sm."""
    sec = ms_per_round / 1e3
    per_el, ipe, captured_on = counters_for(tag, kernel)
    alu_peak = SM_COUNT * SCHEDULERS_PER_SM * (sm_max_mhz or 1965) / 1e3           # G warp instructions / s
    achieved = None if ipe is None else ipe * elements / sec / 1e9
    traffic = None if per_el is None else per_el * elements                         # per launch of rounds_per_launch rounds
    out = {"bound": "alu", "achieved": achieved, "peak": alu_peak, "unit": "Gwarp-inst/s",
           "frac": None if achieved is None else achieved / alu_peak, "traffic": traffic,
           "peak_kind": "148 SMs x 4 schedulers x 1 warp instruction per clock x clocks.max.sm", "kernel": kernel,
           "rounds_per_launch": rounds_per_launch, "warp_inst_per_element_round": ipe,
           "bytes_per_launch": UNIQUE_FRACTION * bpe * elements,
           "replica_GBs": bpe * elements / sec / 1e9, "hbm_peak": peak, "hbm_peak_kind": f"of {peak_kind}"}
    if kernel_source_hash() == NCU_HASH and (tag, kernel) in NCU_PIPES:
        out["pipes_busy"] = NCU_PIPES[(tag, kernel)]
    if traffic is not None:
        dram = traffic / (sec * rounds_per_launch) / 1e9
        out.update({"dram_GBs": dram, "dram_frac_of_measured": dram / peak, "dram_frac_of_8TBs": dram / NOMINAL_HBM_GBS,
                    "traffic_captured_on": captured_on})
    return out


class Timer:
    """CUDA-event timing of netmax_round on the context's stream."""

    def __init__(self, torch, stream, barrier):
        self.torch, self.stream, self.barrier = torch, stream, barrier
        self.start = torch.cuda.Event(enable_timing=True)
        self.stop = torch.cuda.Event(enable_timing=True)

    def rounds(self, g, n):
        self.barrier()
        with self.torch.cuda.stream(self.stream):
            self.start.record()
        g.round(n)
        with self.torch.cuda.stream(self.stream):
            self.stop.record()
        self.stop.synchronize()
        return self.start.elapsed_time(self.stop)

    def repeats(self, g, n, reps=5):
        return [self.rounds(g, n) / n for _ in range(reps)]


def launch_shape(g, rounds, ring):
    """Names the launch shape netmax_round chose, from the number of launches `rounds` rounds took."""
    before = g.kernel_launches
    g.round(rounds)
    per = rounds / max(1, g.kernel_launches - before - (rounds + ring - 1) // ring)      # sampler launches excluded
    if per > 8.5 or (per > 1.5 and g.M * g.d < (1 << 23)):      # (short vectors never take the tile-resident shapes)
        return "all rounds of a call on shared-memory-resident columns", "resident_rounds_kernel", per
    if per > 1.5:
        if g.M > 36:        # more rows than one CTA's slabs hold: the tile is resident across a cluster of CTAs
            return "%d rounds per launch over tiles resident across a thread-block cluster" % round(per), "cluster_rounds_kernel", per
        return "%d rounds per launch over resident tiles" % round(per), "fused_rounds_kernel", per
    return "one launch per round", "round_kernel", per


def measure_config(torch, binding, wk, args, local, timer, peak, peak_kind, sm_max_mhz):
    """One entry of the line's `configs`: the workload in the launch shape the library picks (and, where
    that fuses rounds, one launch per round as well), timed over at least 200 rounds per repeat."""
    speeds = wk.link_speeds(0)
    t_iter, adj = binding.netmax_iteration_times(speeds, wk.d)
    generate = binding.netmax_policy_generate_device if wk.M >= 512 else binding.netmax_policy_generate
    P, rho, _ = generate(t_iter, adj, wk.lr, wk.K, wk.R)
    bf16 = args.storage == "bf16"
    bpe = BYTES_PER_ELEMENT_BF16 if bf16 else BYTES_PER_ELEMENT
    ring = 1024
    g = binding.Netmax(M=wk.M, d=wk.d, lr=wk.lr, link_speed_gbps=speeds, prob=P, rho=rho, sigma=wk.sigma,
                       x0_std=wk.x0_std, c_std=wk.c_std, objective=1, seed=wk.seed, device=local,
                       stream=timer.stream.cuda_stream, trace_rounds=ring, storage=args.storage)
    elements = wk.M * wk.d
    tag = wk.name + ("/bf16" if bf16 else "")
    rounds = 200 if elements > 1 << 22 else 2000
    shape, kernel, per = launch_shape(g, 24, ring)
    g.round(20)
    ms = timer.repeats(g, rounds, 3)
    best = min(ms)
    entry = {"M": wk.M, "d": wk.d, "launch_shape": shape, "rounds_timed": rounds, "ms_per_round": best,
             "ms_per_round_median": statistics.median(ms), "rounds_per_s": 1e3 / best,
             "replica_GBs": bpe * elements / (best / 1e3) / 1e9, "peer_draws_per_s": wk.M * 1e3 / best}
    if kernel == "round_kernel":
        entry["roofline"] = hbm_roofline(tag, kernel, best, elements, bpe, peak, peak_kind)
    else:
        entry["roofline"] = issue_roofline(tag, kernel, best, elements, bpe, per, sm_max_mhz, peak, peak_kind)
    # the sampler alone: batched launches of 1024 rounds x M draws (Algorithm 2's peer selection)
    batch = 1024
    draws = torch.empty((batch, wk.M), dtype=torch.int32, device="cuda")
    for _ in range(3):
        g.sample_peers(0, batch, draws.data_ptr())
    timer.barrier()
    with torch.cuda.stream(timer.stream):
        timer.start.record()
    for rep in range(10):
        g.sample_peers(rep * batch, batch, draws.data_ptr())
    with torch.cuda.stream(timer.stream):
        timer.stop.record()
    timer.stop.synchronize()
    entry["sampler_only_draws_per_s"] = 10 * batch * wk.M / (timer.start.elapsed_time(timer.stop) / 1e3)
    del draws
    if kernel in ("fused_rounds_kernel", "cluster_rounds_kernel"):
        g.set_fuse_rounds(1)
        g.round(20)
        one = min(timer.repeats(g, rounds, 3))
        entry["one_launch_per_round"] = {"ms_per_round": one,
                                         "roofline": hbm_roofline(tag, "round_kernel", one, elements, bpe, peak, peak_kind)}
    g.close()
    torch.cuda.empty_cache()
    return entry


def run_ours(args, w):
    import torch
    import torch.distributed as dist
    from paper_2009_05766_b200 import binding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if world != args.gpus:
        raise SystemExit(f"--gpus {args.gpus} but WORLD_SIZE={world}: launch with torch.distributed.run")

    base = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        base = cpu_baseline(w, storage=args.storage)          # before the first CUDA call

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    binding.lib()

    # control plane (host, untimed): Algorithm 3 on the workload's link speeds
    speeds = w.link_speeds(0)
    t_iter, adj = binding.netmax_iteration_times(speeds, w.d)
    generate = binding.netmax_policy_generate_device if w.M >= 512 else binding.netmax_policy_generate
    P, rho, pinfo = generate(t_iter, adj, w.lr, w.K, w.R)

    bf16 = args.storage == "bf16"
    bytes_per_element = BYTES_PER_ELEMENT_BF16 if bf16 else BYTES_PER_ELEMENT
    plan = shard_plan(w.d, world, rank, 8 if bf16 else 4)
    stream = torch.cuda.Stream()
    ring = 1024
    size = binding.Netmax.workspace_size(w.M, w.d, ring, storage=args.storage)
    ws = torch.empty(size + 256, dtype=torch.uint8, device="cuda")       # device memory from PyTorch
    ws_ptr = (ws.data_ptr() + 255) // 256 * 256
    g = binding.Netmax(M=w.M, d=w.d, lr=w.lr, link_speed_gbps=speeds, prob=P, rho=rho, sigma=w.sigma,
                       x0_std=w.x0_std, c_std=w.c_std, objective=1, seed=w.seed, device=local,
                       stream=stream.cuda_stream, trace_rounds=ring, workspace=ws_ptr, workspace_bytes=size,
                       element_offset=plan["element_offset"], storage=args.storage, fuse_rounds=args.fuse_rounds)

    def barrier():
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    elements = w.M * w.d
    timer = Timer(torch, stream, barrier)
    start, stop = timer.start, timer.stop

    g.round(args.warmup)
    barrier()
    launches0 = g.kernel_launches
    with ClockSampler(local) as clocks:
        ms = timer.rounds(g, args.steps)                      # the contract's timed region: exactly K steps
        launches = g.kernel_launches - launches0
        barrier()
        # repeats of a run long enough to time well (at least 200 rounds each): best and median per round
        rep_rounds = max(200, min(args.steps, 2000)) if elements > 1 << 22 else max(2000, args.steps)
        rep_ms = timer.repeats(g, rep_rounds)
    if world > 1:
        tmax = torch.tensor([ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        ms = float(tmax.item())
    sec = ms / 1e3
    value = bytes_per_element * elements * world * args.steps / sec / 1e9

    rounds_per_launch = args.steps / max(1, launches - (args.steps + ring - 1) // ring)   # sampler launches excluded
    resident = rounds_per_launch > 8.5 or (rounds_per_launch > 1.5 and elements < (1 << 23))   # short vectors: all rounds
    fused = rounds_per_launch > 1.5 and not resident                                          # of a call on resident columns
    single_ms = None
    if fused:                       # the same rounds, one launch each: the HBM-bound kernel
        g.set_fuse_rounds(1)
        g.round(args.warmup)
        single_ms = timer.repeats(g, rep_rounds)
        g.set_fuse_rounds(args.fuse_rounds)

    # end to end through the C ABI with host buffers: upload x and c, one round, download x'
    e2e_steps = max(1, min(args.steps, args.e2e_steps))
    hx = torch.empty((w.M, w.d), dtype=torch.float32, pin_memory=True)
    hc = torch.empty((w.M, w.d), dtype=torch.float32, pin_memory=True)
    ho = torch.empty((w.M, w.d), dtype=torch.float32, pin_memory=True)
    g.read_replicas(hx.data_ptr())
    lib = binding.lib()
    assert lib.netmax_read_centres(g._h, hc.data_ptr()) == 0

    def e2e_step():           # the public call for a step through host buffers: upload, one round, download, pipelined by columns
        g.round_from_host(hx.data_ptr(), hc.data_ptr(), 1, ho.data_ptr(), args.e2e_chunks)

    def e2e_step_serial():    # the same through the four separate calls, one after the other
        g.set_replicas(hx.data_ptr())
        g.set_centres(hc.data_ptr())
        g.round(1)
        g.read_replicas(ho.data_ptr())

    def time_e2e(step):
        for _ in range(2):
            step()
        barrier()
        t0 = time.perf_counter()
        with torch.cuda.stream(stream):
            start.record()
        for _ in range(e2e_steps):
            step()
        with torch.cuda.stream(stream):
            stop.record()
        stop.synchronize()
        return start.elapsed_time(stop), time.perf_counter() - t0

    e2e_serial_ms, _ = time_e2e(e2e_step_serial)
    e2e_ms, e2e_wall = time_e2e(e2e_step)
    if world > 1:
        tmax = torch.tensor([e2e_ms], device="cuda", dtype=torch.float64)
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        e2e_ms = float(tmax.item())
    e2e_value = bytes_per_element * elements * world * e2e_steps / (e2e_ms / 1e3) / 1e9
    del hx, hc, ho

    # the sampler alone: one batched launch of 1024 rounds x M draws (Algorithm 2's peer selection)
    batch = 1024
    draws = torch.empty((batch, w.M), dtype=torch.int32, device="cuda")
    for _ in range(3):
        g.sample_peers(0, batch, draws.data_ptr())
    barrier()
    with torch.cuda.stream(stream):
        start.record()
    for rep in range(10):
        g.sample_peers(rep * batch, batch, draws.data_ptr())
    with torch.cuda.stream(stream):
        stop.record()
    stop.synchronize()
    sampler_draws_per_s = 10 * batch * w.M / (start.elapsed_time(stop) / 1e3)

    cons, loss = g.telemetry(g.rounds_done - 1, 1)
    peak, peak_kind = measured_peak()
    per_round_ms = ms / args.steps
    tag = w.name + ("/bf16" if bf16 else "")
    sm_max_mhz = clocks.summary()["sm_max_mhz"]
    if fused or resident:
        kernel = (("cluster_rounds_kernel" if w.M > 36 else "fused_rounds_kernel") if fused else
                  ("multi_round_kernel" if args.fuse_rounds == 1 else "resident_rounds_kernel"))
        roofline = issue_roofline(tag, kernel, per_round_ms, elements, bytes_per_element, rounds_per_launch, sm_max_mhz,
                                  peak, peak_kind)
    else:
        roofline = hbm_roofline(tag, "round_kernel", per_round_ms, elements, bytes_per_element, peak, peak_kind)
    line = {
        "metric": "replica GB/s", "value": value, "unit": "GB/s", "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": per_round_ms, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16 storage, f32 arithmetic" if bf16 else "f32", "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "d_per_gpu": w.d, "global_d": plan["global_d"], "lr": w.lr,
                   "sigma": w.sigma, "policy": f"Algorithm 3, K={w.K}, R={w.R}, rho={rho:.6g}",
                   "sharding": "columns, no exchange" if world > 1 else "none", "storage": args.storage,
                   "l2": "inputs larger than L2: each of x, x', c is %.0f MB" % (elements * bytes_per_element / 4 / 1e6)},
        "metric_definition": "replica GB/s = 16 bytes (x_i, x_peer, c_i read; x_i' written) x M x d x rounds / time; "
                             "`roofline` holds the fraction of the bound that applies and the DRAM rate from ncu's counters",
        "repeats": {"rounds_each": rep_rounds, "ms_per_step_best": min(rep_ms),
                    "ms_per_step_median": statistics.median(rep_ms)},
        "hbm_footprint_bytes": int(size),
        "rounds_per_s": args.steps / sec, "peer_draws_per_s": w.M * world * args.steps / sec,
        "sampler_only_draws_per_s": sampler_draws_per_s,
        "roofline": roofline,
        "e2e": {"value": e2e_value, "unit": "GB/s", "h2d_bytes_per_step": 2 * elements * 4,
                "d2h_bytes_per_step": elements * 4, "steps": e2e_steps, "ms_per_step": e2e_ms / e2e_steps,
                "wall_ms_per_step": e2e_wall * 1e3 / e2e_steps, "call": "netmax_round_from_host (column chunks pipelined)",
                "ms_per_step_four_separate_calls": e2e_serial_ms / e2e_steps},
        "gpu_launches": int(launches),
        "clocks": clocks.summary(),
        "telemetry_last_round": {"consensus": float(cons[0]), "loss": float(loss[0])},
        "paper_context": "paper: 3.7x/3.4x/1.9x faster convergence than Prague/Allreduce-SGD/AD-PSGD "
                         "(ResNet18, 8x RTX 2080 Ti, throttled 1 GbE); not comparable to this metric",
    }
    if single_ms is not None:
        line["one_launch_per_round"] = {
            "ms_per_step_best": min(single_ms), "ms_per_step_median": statistics.median(single_ms),
            "roofline": hbm_roofline(tag, "round_kernel", min(single_ms), elements, bytes_per_element, peak, peak_kind)}
    if base is not None:
        line["cpu_baseline"] = base
    g.close()
    del ws
    torch.cuda.empty_cache()
    if world == 1 and args.configs != "none" and args.d == 0:
        # every config of the benchmark description in the same process (the headline's own numbers are reused)
        which = [1, 2, 3, 4, 5] if args.configs == "all" else [int(c) for c in args.configs.split(",")]
        configs = {}
        for idx in which:
            wk = workloads.config(idx)
            if wk.name == w.name:
                entry = {"M": w.M, "d": w.d, "launch_shape": "headline (see the top-level keys)",
                         "rounds_timed": rep_rounds, "ms_per_round": min(rep_ms),
                         "ms_per_round_median": statistics.median(rep_ms), "rounds_per_s": 1e3 / min(rep_ms),
                         "replica_GBs": bytes_per_element * elements / (min(rep_ms) / 1e3) / 1e9,
                         "peer_draws_per_s": w.M * 1e3 / min(rep_ms)}
                entry["roofline"] = (issue_roofline(tag, kernel, min(rep_ms), elements, bytes_per_element, rounds_per_launch,
                                                    sm_max_mhz, peak, peak_kind) if (fused or resident) else
                                     hbm_roofline(tag, "round_kernel", min(rep_ms), elements, bytes_per_element, peak, peak_kind))
                if single_ms is not None:
                    entry["one_launch_per_round"] = {"ms_per_round": min(single_ms),
                                                     "roofline": line["one_launch_per_round"]["roofline"]}
                configs["cfg%d" % idx] = entry
                continue
            with ClockSampler(local) as ck:
                entry = measure_config(torch, binding, wk, args, local, timer, peak, peak_kind, sm_max_mhz)
            entry["clocks"] = ck.summary()
            configs["cfg%d" % idx] = entry
        line["configs"] = configs
    if world > 1:
        dist.destroy_process_group()
    if rank == 0:
        print(json.dumps(line), flush=True)


def run_async(args, w):
    """The asynchronous timeline (one worker per global step, Eq. 17): a step is one global step,
    i.e. one replica of d elements updated in place from its peer (16 bytes of HBM per element)."""
    import torch
    from paper_2009_05766_b200 import binding
    if int(os.environ.get("WORLD_SIZE", "1")) != 1 or args.gpus != 1:
        raise SystemExit("--mode async runs on one GPU")
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU path)")
    binding.lib()
    speeds = w.link_speeds(0)
    t_iter, adj = binding.netmax_iteration_times(speeds, w.d)
    P, rho, _ = binding.netmax_policy_generate(t_iter, adj, w.lr, w.K, w.R)
    stream = torch.cuda.Stream()
    g = binding.Netmax(M=w.M, d=w.d, lr=w.lr, link_speed_gbps=speeds, prob=P, rho=rho, sigma=w.sigma,
                       x0_std=w.x0_std, c_std=w.c_std, objective=1, seed=w.seed, stream=stream.cuda_stream,
                       storage=args.storage)
    bytes_per_element = BYTES_PER_ELEMENT_BF16 if args.storage == "bf16" else BYTES_PER_ELEMENT
    g.async_begin(None, 0.9)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    g.async_steps(max(args.warmup, 3) * w.M)
    torch.cuda.synchronize()
    launches0 = g.kernel_launches
    with ClockSampler(0) as clocks:
        with torch.cuda.stream(stream):
            start.record()
        g.async_steps(args.steps)
        with torch.cuda.stream(stream):
            stop.record()
        stop.synchronize()
    ms = start.elapsed_time(stop)
    launches = g.kernel_launches - launches0
    sim_time, steps_done = g.async_time()
    cons, loss = g.measure()
    peak, peak_kind = measured_peak()
    achieved = bytes_per_element * w.d * args.steps / (ms / 1e3) / 1e9
    line = {
        "metric": "replica GB/s", "value": achieved, "unit": "GB/s", "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3) * w.M, "ms_per_step": ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": w.name + ", asynchronous timeline (one worker per global step)", "M": w.M, "d": w.d,
                   "storage": args.storage,
                   "l2": "each replica is %.0f MB; a step touches three of them" % (w.d * bytes_per_element / 4 / 1e6)},
        "global_steps_per_s": args.steps / (ms / 1e3), "steps_per_launch": args.steps / max(launches, 1),
        "simulated_seconds": sim_time,
        "roofline": {"bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                     "traffic": None, "peak_kind": f"of {peak_kind}", "kernel": "step_kernel",
                     "bytes_per_launch": bytes_per_element * w.d * args.steps / max(launches, 1)},
        "gpu_launches": int(launches), "clocks": clocks.summary(),
        "telemetry_now": {"consensus": cons, "loss": loss},
    }
    g.close()
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=20)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--workload", default="cfg2", help="cfg1..cfg5 (default: the ResNet18-sized cfg2)")
    ap.add_argument("--d", type=int, default=0, help="override the workload's vector length (profiling on a smaller case)")
    ap.add_argument("--e2e-steps", type=int, default=5)
    ap.add_argument("--e2e-chunks", type=int, default=0, help="column chunks of the pipelined host round trip (0: automatic)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--configs", default="all",
                    help="one GPU: which of cfg1..cfg5 to time into the line's `configs` (all, none, or e.g. 3,4)")
    ap.add_argument("--fuse-rounds", type=int, default=0,
                    help="rounds per launch over a resident tile: 0 automatic, 1 one launch per round, 2..8")
    ap.add_argument("--storage", choices=["f32", "bf16"], default="f32",
                    help="precision of the replicas in device memory (arithmetic is fp32 either way)")
    ap.add_argument("--mode", choices=["rounds", "async"], default="rounds",
                    help="rounds: synchronous rounds (default); async: the paper's one-worker-per-step timeline")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    w = workloads.config(int(args.workload.replace("cfg", "")))
    if args.d > 0:
        w = w.scaled(d=args.d)
    if args.impl == "reference":
        run_reference(args, w)
    elif args.mode == "async":
        run_async(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
