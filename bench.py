#!/usr/bin/env python
"""Benchmark of libsolgemm's hot path on synthetic data.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference]

One "step" is one pass of the whole hot path -- operand load, tcgen05 contraction, fused epilogue,
store -- over one batch: a single ``sg_gemm`` launch of the GEMM 4096^3 + bias + ReLU problem
(bf16 in, fp32 accumulate, bf16 out).  Rank 0 prints ONE JSON line:

* ``value``      TFLOP/s of the whole job (all ranks), operands resident in HBM, CUDA-event timed,
                 max over ranks; every step uses the next of several distinct buffer sets whose total
                 size exceeds the 126 MB L2, so no step finds its operands left in L2 by the step before.
                 The K timed steps are the K kernel nodes of one CUDA graph (one untimed replay, then the timed
                 one); ``ms_per_step_plain_launches`` is the same K steps launched one by one.
* ``e2e``        the same metric through the public API with pinned HOST buffers: H2D of A, B, bias,
                 the kernel, and D2H of D inside the timed region.
* ``roofline``   the kernel's achieved TFLOP/s against the measured dense-bf16 peak of this machine.
* ``cpu_baseline``  the fp64 CPU oracle, as it stands, timed on a bounded sample of the same problem.
* ``clocks``     SM clock and throttle reasons sampled during the timed region.
* ``per_config`` every one of the five benchmark configurations: kernel-only time (median and best of several
                 repetitions of a CUDA graph over distinct buffer sets), TFLOP/s, algorithmic GB/s, fraction of the
                 Speed-of-Light bound against the measured and the datasheet peaks, the launch plan, the kernel the
                 library ran, the SM clock counted inside it, and torch's library kernels on the same buffers.
* ``c2_burst`` / ``c2_sustained``  the headline problem from an idle GPU (a few launches) and over >= 0.6 s of
                 back-to-back launches (held at the board's power cap), side by side.
* ``kernels_in_timed_region``  the kernel names launched by the timed steps (the library's own record).

``--impl reference`` times the CPU oracle alone (it is this project's reference implementation).
With N > 1 (under torchrun) ``value`` has every rank run the whole problem on its own GPU (replicas, "weak" scaling,
no collective on the data path); ``per_config`` has every rank run its shard of each problem -- rows of A/D, batch
entries, images, whole groups -- timed as the max over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "TFLOP/s and % of SOL (max of FLOP/peak, bytes/HBM) per config at 1 B200"
WORKLOAD = "c2_gemm_4096_bias_relu"
L2_BYTES = 126 * 1024 * 1024
SPEC_PEAK_FLOPS = 2250e12      # NVIDIA B200 dense bf16 (datasheet)
SPEC_PEAK_BW = 8000e9          # NVIDIA B200 HBM3e (datasheet)
PER_CLOCK_FLOPS = 8192.0 * 148  # dense bf16 FLOP per SM clock of the whole chip (148 SMs x 8192 FLOP/clk)
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}
# DRAM bytes per launch (dram__bytes_read.sum + dram__bytes_write.sum) of the dominant kernel, from one ncu capture of
# the timed launch (read + write of one c2 launch); not re-measured by this script.
NCU_DRAM_BYTES_PER_LAUNCH = 71_833_344 + 15_188_736
NCU_DRAM_SOURCE = ("one ncu capture (--metrics dram__bytes_read.sum,dram__bytes_write.sum, one launch) of this kernel, "
                   "sg::contract_kernel<256, true, 0, 4, 1>, on this problem; not re-measured by this run")


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            return json.load(f), "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """Samples SM clock and throttle reasons in a background thread (NVML; read-only)."""

    REASONS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap",
               0x80: "hw_power_brake_slowdown"}

    def __init__(self, index: int, period_s: float = 0.01):
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._thread = None
        self._h = None
        try:
            import pynvml
            pynvml.nvmlInit()
            self._nv = pynvml
            self._h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self._h, pynvml.NVML_CLOCK_SM))
        except Exception:
            self._h = None
        self._period = period_s

    def sample_once(self):
        if self._h is None:
            return
        try:
            self.samples.append(int(self._nv.nvmlDeviceGetClockInfo(self._h, self._nv.NVML_CLOCK_SM)))
            mask = int(self._nv.nvmlDeviceGetCurrentClocksEventReasons(self._h)) \
                if hasattr(self._nv, "nvmlDeviceGetCurrentClocksEventReasons") \
                else int(self._nv.nvmlDeviceGetCurrentClocksThrottleReasons(self._h))
            for bit, name in self.REASONS.items():
                if mask & bit:
                    self.reasons.add(name)
        except Exception:
            pass

    def _run(self):
        while not self._stop.is_set():
            self.sample_once()
            self._stop.wait(self._period)

    def start(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()

    def stop(self) -> dict:
        self._stop.set()
        if self._thread:
            self._thread.join()
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2] if s else None, "sm_max_mhz": self.max_mhz, "samples": len(s),
                "reasons": sorted(self.reasons)}


def physical_gpu_index(local_index: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_index])
        except Exception:
            return local_index
    return local_index


# ------------------------------------------------------------------------------------------ reference arm (CPU oracle)

def oracle_rows_for(seconds: float, hA, hB, hb, epi: str, M: int):
    """Pick a row count whose oracle run lasts about `seconds`, from a short pilot. Returns (rows, rows_per_s)."""
    from oracle import oracle as orc
    pilot = 8
    t0 = time.perf_counter()
    orc.gemm(hA, hB, bias=hb, epi=epi, rows=(0, pilot))
    rate = pilot / max(time.perf_counter() - t0, 1e-6)
    rows = int(max(1, min(M, rate * seconds)))
    return rows, rate


def run_reference(args, rank: int, world: int) -> None:
    if rank != 0:
        return
    import torch
    from oracle import oracle as orc
    from paper_2603_29010_b200 import inputs
    c = inputs.CONFIGS[WORKLOAD]
    M, N, K = c["M"], c["N"], c["K"]
    hA, hB, hb = inputs.make_gemm(M, N, K, c["dist"], c["scale"], bias=True)
    total = max(args.steps + args.warmup, 1)
    per_step_s = min(15.0, 150.0 / total)
    rows, _ = oracle_rows_for(per_step_s, hA, hB, hb, c["epi"], M)
    for _ in range(args.warmup):
        orc.gemm(hA, hB, bias=hb, epi=c["epi"], rows=(0, rows))
    t0 = time.perf_counter()
    for s in range(args.steps):
        r0 = (s * rows) % max(M - rows + 1, 1)
        orc.gemm(hA, hB, bias=hb, epi=c["epi"], rows=(r0, r0 + rows))
    dt = time.perf_counter() - t0
    flops = 2.0 * rows * N * K * args.steps
    value = flops / dt / 1e12
    cores = orc.num_threads()
    sample = f"{rows} of {M} output rows per step ({rows * N} of {M * N} elements), all N and K"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": "TFLOP/s", "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / max(args.steps, 1) * 1e3,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD, "M": M, "N": N, "K": K, "layout": "A row-major, B column-major",
                       "epilogue": "bias+relu", "accumulate": "fp64", "out": "fp64 (unrounded)",
                       "note": "CPU oracle (plain fp64 loops, OpenMP over rows), timed as it stands on a bounded sample"},
            "cpu_baseline": {"value": value, "unit": "TFLOP/s", "cores": cores, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": "TFLOP/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


# ------------------------------------------------------------------------------------------ our arm

def time_steps(fn, steps: int, torch) -> float:
    """Seconds for `steps` calls of fn(i) on the current stream, CUDA-event timed."""
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    start.record()
    for i in range(steps):
        fn(i)
    stop.record()
    stop.synchronize()
    return start.elapsed_time(stop) * 1e-3


def _median(xs):
    s = sorted(xs)
    return s[len(s) // 2]


def time_graph_repeats(fns, torch, launches_wanted: int, repeats: int, idle_s: float = 0.03):
    """Per-launch seconds of `repeats` timed repetitions.  One CUDA graph holds one launch per buffer set (the sets
    together exceed the L2, so no launch finds its operands left there by the launch before); a repetition replays it
    back to back until about `launches_wanted` launches have run (a few milliseconds: a burst, like the measurement
    behind the burst peak it is compared with), CUDA-event timed on the launching stream."""
    for f in fns[:min(3, len(fns))]:
        f()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for f in fns:
            f()
    replays = max(1, -(-launches_wanted // len(fns)))
    for _ in range(3):
        graph.replay()
    torch.cuda.synchronize()
    out = []
    for _ in range(repeats):
        torch.cuda.synchronize()
        time.sleep(idle_s)                      # every repetition starts from a settled, idle GPU (a short burst)
        graph.replay()                          # one untimed pass wakes the clocks
        out.append(time_steps(lambda i: graph.replay(), replays, torch) / (replays * len(fns)))
    return out, replays * len(fns), graph


def config_workloads(sg, inputs, sharding, torch, dev, rank: int, world: int):
    """The five benchmark configurations as (name, launch closures over distinct buffer sets, SOL arguments of this
    rank's shard, torch-library closure, note).  With world > 1 every rank gets its shard of each problem (rows of A/D,
    batch entries, images, whole groups); with world == 1 the shard is the whole problem."""
    import torch.nn.functional as F
    C = inputs.CONFIGS
    bf = torch.bfloat16
    work = []

    # c1: one 256^3 product.  Too small to shard (two tile rows): every rank runs it whole.
    c = C["c1_gemm_256"]
    sets = 400                                             # 400 x 393 KB = 157 MB > L2
    A1, B1, _ = inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"], device=dev, batch=sets)
    O1 = torch.empty(sets, c["M"], c["N"], dtype=bf, device=dev)
    work.append(dict(name="c1_gemm_256", fns=[(lambda i=i: sg.gemm(A1[i], B1[i], out=O1[i])) for i in range(sets)],
                     sol=dict(op="gemm", M=c["M"], N=c["N"], K=c["K"]), launches=800,
                     lib=lambda: torch.matmul(A1[0], B1[0].t()), partition="replicated (not sharded)",
                     keep=(A1, B1, O1)))

    # c2: rows of A and D
    c = C["c2_gemm_4096_bias_relu"]
    r0, r1 = sharding.gemm_rows(c["M"], world, rank, 256)
    sets = 7
    d2 = [inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"], bias=True, seed=inputs.BASE_SEED + i, device=dev)
          for i in range(sets)]
    O2 = [torch.empty(r1 - r0, c["N"], dtype=bf, device=dev) for _ in range(sets)]
    epi2 = c["epi"]
    work.append(dict(name="c2_gemm_4096_bias_relu",
                     fns=[(lambda i=i: sg.gemm(d2[i][0][r0:r1], d2[i][1], bias=d2[i][2], out=O2[i], epi=epi2)) for i in range(sets)],
                     sol=dict(op="gemm", M=r1 - r0, N=c["N"], K=c["K"], has_bias=1), launches=28,
                     lib=lambda: torch.relu(torch.addmm(d2[0][2], d2[0][0][r0:r1], d2[0][1].t())),
                     partition=f"rows {r0}:{r1} of A and D, B replicated", keep=(d2, O2)))

    # c3: batch entries
    c = C["c3_batched_128x256x256x512_gelu"]
    b0, b1 = sharding.batch_entries(c["batch"], world, rank)
    sets = 8                                               # 8 x 84 MB > L2
    d3 = [inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"], seed=inputs.BASE_SEED + i, device=dev, batch=c["batch"])
          for i in range(sets)]
    O3 = [torch.empty(b1 - b0, c["M"], c["N"], dtype=bf, device=dev) for _ in range(sets)]
    epi3 = c["epi"]
    work.append(dict(name="c3_batched_128x256x256x512_gelu",
                     fns=[(lambda i=i: sg.batched_gemm(d3[i][0][b0:b1], d3[i][1][b0:b1], out=O3[i], epi=epi3)) for i in range(sets)],
                     sol=dict(op="batched", M=c["M"], N=c["N"], K=c["K"], batch_or_groups=b1 - b0), launches=160,
                     lib=lambda: F.gelu(torch.bmm(d3[0][0][b0:b1], d3[0][1][b0:b1].transpose(1, 2)), approximate="tanh"),
                     partition=f"batch entries {b0}:{b1}", keep=(d3, O3)))

    # c4: images
    c4 = C["c4_conv_32x56x56x256_k256_3x3_bias_relu"]
    n0, n1 = sharding.conv_images(c4["N"], world, rank)
    sets = 4                                               # 4 x 104 MB > L2
    d4 = [inputs.make_conv(c4["N"], c4["H"], c4["W"], c4["C"], c4["K"], c4["R"], c4["S"], c4["dist"], c4["scale"],
                           bias=True, seed=inputs.BASE_SEED + i, device=dev) for i in range(sets)]
    O4 = [torch.empty(n1 - n0, 56, 56, c4["K"], dtype=bf, device=dev) for _ in range(sets)]
    geo = {k: c4[k] for k in ("N", "H", "W", "C", "K", "R", "S", "pad")}
    geo["N"] = n1 - n0
    work.append(dict(name="c4_conv_32x56x56x256_k256_3x3_bias_relu",
                     fns=[(lambda i=i: sg.conv2d_fprop(d4[i][0][n0:n1], d4[i][1], pad=c4["pad"], bias=d4[i][2], out=O4[i],
                                                       epi=c4["epi"])) for i in range(sets)],
                     sol=dict(op="conv2d", conv=geo, has_bias=1), launches=32,
                     lib=lambda: torch.relu(F.conv2d(d4[0][0][n0:n1].permute(0, 3, 1, 2), d4[0][1].permute(0, 3, 1, 2), d4[0][2],
                                                     padding=1)),
                     partition=f"images {n0}:{n1}, filter replicated", keep=(d4, O4)))

    # c5: whole groups, largest first onto the lightest rank
    c5 = C["c5_grouped_16xMx4096x4096_silu"]
    Ms_all = inputs.grouped_sizes(c5["groups"], c5["M_lo"], c5["M_hi"])
    mine = sharding.assign_groups(Ms_all, world)[rank]
    Ms = [Ms_all[g] for g in mine]
    As, Bs = inputs.make_grouped(Ms_all, c5["N"], c5["K"], c5["dist"], c5["scale"], device=dev)     # 1.1 GB > L2
    As, Bs = [As[g] for g in mine], [Bs[g] for g in mine]
    O5 = [torch.empty(m, c5["N"], dtype=bf, device=dev) for m in Ms]
    ws = torch.empty(sg.grouped_workspace_size(max(len(Ms), 1)), dtype=torch.uint8, device=dev)
    work.append(dict(name="c5_grouped_16xMx4096x4096_silu",
                     fns=[lambda: sg.grouped_gemm(As, Bs, outs=O5, epi=c5["epi"], workspace=ws)] if Ms else [],
                     sol=dict(op="grouped", N=c5["N"], K=c5["K"], batch_or_groups=len(Ms), Ms=Ms), launches=4,
                     lib=lambda: [F.silu(a @ b.t()) for a, b in zip(As, Bs)],
                     partition=f"groups {mine} (M_i {Ms})", keep=(As, Bs, O5, ws), extra={"M_i": Ms_all}))
    return work


def bench_per_config(sg, inputs, sharding, torch, dist, dev, peaks, rank: int, world: int, repeats: int = 9,
                     torch_ref: bool = True) -> dict:
    """Kernel-only timing of every benchmark configuration (this rank's shard; max over ranks), median and best of
    `repeats` repetitions, beside the Speed-of-Light bound of the WHOLE problem, the launch plan, the kernel the library
    ran, the SM clock counted inside it, and -- on one GPU -- torch's library kernels on the same buffers."""
    out = {}
    hw = dict(peak_flops=peaks["bf16_tflops"] * 1e12, peak_bytes_per_s=peaks["hbm_gbs"] * 1e9)
    spec = dict(peak_flops=SPEC_PEAK_FLOPS, peak_bytes_per_s=SPEC_PEAK_BW)
    for w in config_workloads(sg, inputs, sharding, torch, dev, rank, world):
        name = w["name"]
        if w["fns"]:
            times, launches, graph = time_graph_repeats(w["fns"], torch, w["launches"], repeats)
            mhz = sg.last_kernel_clock_mhz()
            plan, kernel = sg.last_launch_plan(), sg.last_kernel_name()
            if "contract_kernel" not in kernel:
                mhz = 0.0                      # only the contraction kernel counts its own clock
            del graph
            # the warm regime: the same launch on ONE buffer set, back to back (operands the L2 can hold stay there)
            warm_times, _, graph = time_graph_repeats([w["fns"][0]] * min(8, max(2, len(w["fns"]))), torch, w["launches"], 5)
            del graph
        else:
            times, launches, mhz, plan, kernel, warm_times = [0.0] * repeats, 0, 0.0, {}, "", [0.0]
        med, best, warm = _median(times), min(times), _median(warm_times)
        if world > 1:
            t = torch.tensor([med, best, warm], dtype=torch.float64, device=dev)
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
            med, best, warm = float(t[0]), float(t[1]), float(t[2])
        # bound of the whole problem (all ranks' shards together)
        whole = dict(w["sol"])
        c = inputs.CONFIGS[name]
        if name.startswith("c2"):
            whole["M"] = c["M"]
        elif name.startswith("c3"):
            whole["batch_or_groups"] = c["batch"]
        elif name.startswith("c4"):
            whole["conv"] = dict(whole["conv"], N=c["N"])
        elif name.startswith("c5"):
            whole["Ms"] = w["extra"]["M_i"]
            whole["batch_or_groups"] = len(whole["Ms"])
        copies = world if name.startswith("c1") else 1
        sol_m, sol_s = sg.sol_bound(**whole, **hw), sg.sol_bound(**whole, **spec)
        clock_peak = PER_CLOCK_FLOPS * mhz * 1e6 if mhz else 0.0
        rec = {"us": med * 1e6, "us_best": best * 1e6, "us_warm_l2": warm * 1e6, "repeats": repeats, "launches_per_repeat": launches,
               "tflops": copies * sol_m["flops"] / med / 1e12, "gbs": copies * sol_m["bytes"] / med / 1e9,
               "flops": sol_m["flops"], "bytes": sol_m["bytes"],
               "bound": "tensor" if sol_m["compute_bound"] else "hbm",
               "t_sol_measured_us": sol_m["t_sol_s"] * 1e6, "frac_of_sol_measured": sol_m["t_sol_s"] / med / (world if copies == 1 else 1),
               "t_sol_spec_us": sol_s["t_sol_s"] * 1e6, "frac_of_sol_spec": sol_s["t_sol_s"] / med / (world if copies == 1 else 1),
               "sm_mhz_in_kernel": round(mhz, 1) if mhz else None, "tiling": plan, "kernel": kernel, "buffer_sets": len(w["fns"]),
               "partition": w["partition"] if world > 1 else "whole problem",
               "timing": "CUDA graph of one launch per buffer set (sets exceed L2), replayed for ~3 ms after 30 ms idle; us = median, us_best = best of the repeats; "
                         "us_warm_l2 = the same protocol on one buffer set (median of 5): context, never the reported number"}
        if sol_m["compute_bound"] and clock_peak:
            rec["frac_of_per_clock_tensor_peak"] = sol_m["flops"] / med / clock_peak / (world if copies == 1 else 1)
        rec["suspicious_faster_than_0.9_sol_spec"] = bool(med * (world if copies == 1 else 1) < 0.9 * sol_s["t_sol_s"])
        rec.update(w.get("extra", {}))
        if torch_ref and world == 1 and w["fns"]:
            lib = w["lib"]
            for _ in range(3):
                lib()
            torch.cuda.synchronize()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g):
                lib()
            g.replay()
            torch.cuda.synchronize()
            reps = max(3, min(200, int(2e-3 / max(med, 1e-6))))
            rec["torch_library_us"] = _median([time_steps(lambda i: g.replay(), reps, torch) / reps for _ in range(3)]) * 1e6
            rec["torch_library_note"] = "torch's library kernels (unfused epilogue where torch has none) on one warm buffer set: context, not a target"
            del g
            if not sol_m["compute_bound"] and sol_m["bytes"] >= (1 << 20):
                # what a plain device copy moving the same number of bytes costs per launch under the same protocol
                # (start and end of a launch included): the practical floor of a launch bound by memory traffic
                half = int(sol_m["bytes"]) // 2
                pairs = max(2, -(-2 * L2_BYTES // (2 * half)) + 1)
                src = [torch.empty(half, dtype=torch.uint8, device=dev) for _ in range(pairs)]
                dst = [torch.empty(half, dtype=torch.uint8, device=dev) for _ in range(pairs)]
                ct, _, g = time_graph_repeats([(lambda i=i: dst[i].copy_(src[i])) for i in range(pairs)], torch, w["launches"], 5)
                rec["device_copy_same_bytes_us"] = _median(ct) * 1e6
                rec["frac_of_device_copy_same_bytes"] = _median(ct) / med
                del g, src, dst
        out[name] = rec
        del w
        torch.cuda.empty_cache()
    return out


def bench_shape_sweep(sg, torch, dev) -> dict:
    """The GEMM shape classes of the paper's workload list (square, LLM-like, small and large K, irregular, tall-skinny,
    matrix-vector, a few rows against a weight matrix, batched) through this library and, for context, through
    torch.matmul / torch.bmm (library kernels), each as one CUDA graph over rotating buffer sets."""
    bf = torch.bfloat16
    out = {}

    def time_graph(fns, reps=10):
        for f in fns[:2]:
            f()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for f in fns:
                f()
        graph.replay()
        torch.cuda.synchronize()
        best = float("inf")
        for _ in range(3):
            best = min(best, time_steps(lambda i: graph.replay(), reps, torch) / (reps * len(fns)))
        return best

    def run(M, N, K, batch=1):
        nbytes = batch * (M * K + N * K + M * N) * 2
        sets = max(1, min(8, int(300e6 // nbytes) + 1))
        shape = (lambda r, c: (r, c)) if batch == 1 else (lambda r, c: (batch, r, c))
        As = [torch.randn(*shape(M, K), device=dev).to(bf) for _ in range(sets)]
        Bs = [torch.randn(*shape(N, K), device=dev).to(bf) for _ in range(sets)]
        Os = [torch.empty(*shape(M, N), dtype=bf, device=dev) for _ in range(sets)]
        if batch == 1:
            t = time_graph([(lambda i=i: sg.gemm(As[i], Bs[i], out=Os[i])) for i in range(sets)])
            plan = sg.last_launch_plan()
            tl = time_graph([(lambda i=i: torch.matmul(As[i], Bs[i].t(), out=Os[i])) for i in range(sets)])
        else:
            t = time_graph([(lambda i=i: sg.batched_gemm(As[i], Bs[i], out=Os[i])) for i in range(sets)])
            plan = sg.last_launch_plan()
            tl = time_graph([(lambda i=i: torch.bmm(As[i], Bs[i].transpose(1, 2), out=Os[i])) for i in range(sets)])
        flops = 2.0 * batch * M * N * K
        out[f"b{batch}_{M}x{N}x{K}"] = {"us": round(t * 1e6, 2), "tflops": round(flops / t / 1e12, 1), "gbs": round(nbytes / t / 1e9),
                                        "library_us": round(tl * 1e6, 2), "library_over_ours": round(tl / t, 2),
                                        "buffer_sets": sets, "plan": plan}

    for shp in [(4096, 4096, 4096), (2048, 4096, 8192), (8192, 8192, 8192), (16384, 16384, 32), (16384, 16384, 64), (8192, 8192, 128),
                (8192, 8192, 256), (256, 256, 131072), (4096, 4096, 14336), (4096, 14336, 4096), (2047, 2040, 2056), (1000, 1000, 1000),
                (3000, 5000, 7000), (32768, 64, 4096), (32768, 128, 1024), (64, 32768, 4096), (512, 512, 512), (1024, 1024, 1024),
                (2048, 2048, 2048), (8192, 1024, 8192), (1024, 8192, 8192),
                (8192, 1, 8192), (4096, 1, 4096), (1, 8192, 8192), (1, 11008, 4096), (2, 8192, 8192), (4, 8192, 8192), (4, 4096, 14336),
                (8, 4096, 14336), (16, 8192, 8192), (32, 4096, 4096), (64, 8192, 8192), (64, 14336, 4096), (128, 8192, 8192)]:
        run(*shp)
    for shp in [(512, 512, 64, 128), (512, 64, 512, 128), (2048, 2048, 128, 32), (2048, 128, 2048, 32), (128, 128, 128, 1024),
                (1024, 1024, 1024, 16)]:
        run(*shp)
    return out


def bench_widened(sg, inputs, torch, dev, peaks) -> dict:
    """Kernel-only timings of the rows built beyond the five configurations: residual and extended epilogues, other
    input types and operand layouts, skinny long-K shapes, the transpose stage and the convolution gradients."""
    out = {}
    hw = dict(peak_flops=peaks["bf16_tflops"] * 1e12, peak_bytes_per_s=peaks["hbm_gbs"] * 1e9)

    def timed(name, fns, sol_kw, reps=20, note=None):
        for f in fns[:2]:
            f()
        torch.cuda.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            for f in fns:
                f()
        graph.replay()
        torch.cuda.synchronize()
        dt = time_steps(lambda i: graph.replay(), reps, torch) / (reps * len(fns))
        sol = sg.sol_bound(**sol_kw, **hw)
        out[name] = {"us": round(dt * 1e6, 2), "tflops": round(sol["flops"] / dt / 1e12, 1), "gbs": round(sol["bytes"] / dt / 1e9),
                     "frac_of_sol_measured_bf16_peaks": round(sol["t_sol_s"] / dt, 3), "plan": sg.last_launch_plan()}
        if note:
            out[name]["note"] = note

    n = 4096
    sets = 7
    bf = torch.bfloat16
    data = [inputs.make_gemm(n, n, n, "normal", 1 / 64., bias=True, seed=i, device=dev) for i in range(sets)]
    outs = [torch.empty(n, n, dtype=bf, device=dev) for _ in range(sets)]
    res = [inputs.normal([n, n], 90 + i, 3, device=dev) for i in range(2)]
    gemm_sol = dict(op="gemm", M=n, N=n, K=n, has_bias=1)
    timed("gemm4096_bias_relu", [(lambda i=i: sg.gemm(*data[i][:2], bias=data[i][2], out=outs[i], epi="relu")) for i in range(sets)],
          gemm_sol)
    timed("gemm4096_bias_relu_residual_beta1",
          [(lambda i=i: sg.gemm(*data[i][:2], bias=data[i][2], C=res[i % 2], beta=1.0, out=outs[i], epi="relu")) for i in range(sets)],
          dict(gemm_sol, beta=1.0))
    rs = torch.rand(n, device=dev) + 0.5
    cs = torch.rand(n, device=dev) + 0.5
    aux = torch.empty(n, n, dtype=bf, device=dev)
    timed("gemm4096_ex_scales_gelu_auxstore_residual",
          [(lambda i=i: sg.gemm(*data[i][:2], bias=data[i][2], out=outs[i], epi="gelu",
                                ex=dict(row_scale=rs, col_scale=cs, aux_store=aux, aux_load=res[i % 2], post_scale=0.5)))
           for i in range(sets)], gemm_sol, note="bytes of the scales and aux tensors not counted in the bound")
    for la, lb in (("col", "col"), ("row", "row"), ("col", "row")):
        timed(f"gemm4096_layout_A{la}_B{lb}",
              [(lambda i=i: sg.gemm(data[i][0], data[i][1], out=outs[i], layout_a=la, layout_b=lb)) for i in range(sets)],
              dict(op="gemm", M=n, N=n, K=n))
    h16 = [(data[i][0].to(torch.float16), data[i][1].to(torch.float16)) for i in range(sets)]
    o16 = [torch.empty(n, n, dtype=torch.float16, device=dev) for _ in range(2)]
    timed("gemm4096_fp16_in_fp16_out", [(lambda i=i: sg.gemm(*h16[i], out=o16[i % 2])) for i in range(sets)], dict(op="gemm", M=n, N=n, K=n))
    del h16, o16
    f32 = [(data[i][0].float(), data[i][1].float()) for i in range(4)]
    o32 = [torch.empty(n, n, dtype=torch.float32, device=dev) for _ in range(2)]
    timed("gemm4096_fp32_in_tf32_fp32_out", [(lambda i=i: sg.gemm(*f32[i], out=o32[i % 2])) for i in range(4)],
          dict(op="gemm", M=n, N=n, K=n, elem_bytes_in=4, elem_bytes_out=4),
          note="the paper's worked SOL example (4096^3, fp32 tensors, TF32 tensor cores); fraction against the bf16 peak: "
               "the tf32 rate is half of it")
    del f32, o32
    for dt8, nm in ((torch.float8_e4m3fn, "e4m3"), (torch.float8_e5m2, "e5m2")):
        q = [(data[i][0].float().mul(64).to(dt8), data[i][1].float().mul(64).to(dt8)) for i in range(sets)]
        timed(f"gemm4096_fp8_{nm}_in_bf16_out", [(lambda i=i: sg.gemm(*q[i], out=outs[i])) for i in range(sets)],
              dict(op="gemm", M=n, N=n, K=n, elem_bytes_in=1), note="fraction against the bf16 peak: above 1 is expected")
        del q
    q8 = [(data[i][0].float().mul(2048).clamp(-127, 127).to(torch.int8), data[i][1].float().mul(2048).clamp(-127, 127).to(torch.int8))
          for i in range(sets)]
    timed("gemm4096_int8_in_bf16_out", [(lambda i=i: sg.gemm(*q8[i], out=outs[i], alpha=2.0 ** -22)) for i in range(sets)],
          dict(op="gemm", M=n, N=n, K=n, elem_bytes_in=1), note="integer tensor-core path; fraction against the bf16 peak")
    del q8
    del data, outs, res, aux
    for (M, N, K) in ((256, 256, 32768), (512, 512, 16384), (128, 4096, 16384), (2048, 4096, 8192), (8192, 8192, 8192)):
        A = inputs.normal([M, K], 1, 1, K ** -0.5, device=dev)
        B = inputs.normal([N, K], 1, 2, 1.0, device=dev)
        O = torch.empty(M, N, dtype=bf, device=dev)
        timed(f"gemm_{M}x{N}x{K}", [lambda: sg.gemm(A, B, out=O)], dict(op="gemm", M=M, N=N, K=K), reps=10,
              note="one buffer set (operands may stay in L2)")
        del A, B, O
    # the three-stage layout pipeline around the benchmark convolution: fp32 NCHW in, fp32 NCHW out
    xs = [torch.randn(32, 256, 56, 56, device=dev) / 48 for _ in range(3)]
    wf = inputs.make_conv(32, 56, 56, 256, 256, 3, 3, "normal", 1 / 48.0, bias=True, seed=3, device=dev)
    timed("pipeline_nchw_fp32_conv3x3_nchw_fp32_32x256x56x56",
          [(lambda i=i: sg.conv2d_fprop_nchw(xs[i], wf[1], pad=(1, 1), bias=wf[2], epi="relu")) for i in range(3)],
          dict(op="conv2d", conv=dict(N=32, H=56, W=56, C=256, K=256, R=3, S=3, pad=(1, 1))),
          note="three launches (transpose + convert, convolution, transpose + convert); the bound is the convolution's alone")
    del xs, wf
    # matrix-vector products (N = 1): a stream over the matrix, several matrices in turn so that none stays in the L2
    for (R, K) in ((4096, 4096), (11008, 4096), (8192, 8192), (256, 131072), (16384, 16384)):
        nset = max(2, min(12, int(400e6 // (R * K * 2)) + 1))
        Ws = [torch.randn(R, K, device=dev).to(bf) for _ in range(nset)]
        x = torch.randn(1, K, device=dev).to(bf)
        ys = [torch.empty(R, 1, dtype=bf, device=dev) for _ in range(nset)]
        timed(f"gemv_{R}x{K}", [(lambda i=i: sg.gemm(Ws[i], x, out=ys[i])) for i in range(nset)], dict(op="gemm", M=R, N=1, K=K),
              note="plan: rows per CTA in 'tiles', K ranges in 'tail_split' (negative), CTAs in 'grid'")
        del Ws, x, ys
    for (b, r, c_) in ((32, 256, 3136), (8, 4096, 4096)):
        for di, do in ((torch.float32, bf), (bf, bf)):
            xs = [torch.randn(b, r, c_, device=dev).to(di) for _ in range(4)]
            ys = [torch.empty(b, c_, r, dtype=do, device=dev) for _ in range(4)]
            timed(f"transpose_{b}x{r}x{c_}_{str(di)[6:]}_to_{str(do)[6:]}", [(lambda i=i: sg.transpose(xs[i], out=ys[i])) for i in range(4)],
                  dict(op="transpose", transpose_shape=(b, r, c_), transpose_dtypes=(di, do)))
            del xs, ys
    cv = inputs.CONFIGS["c4_conv_32x56x56x256_k256_3x3_bias_relu"]
    geo = {k: cv[k] for k in ("N", "H", "W", "C", "K", "R", "S", "pad")}
    X = [inputs.normal([cv["N"], cv["H"], cv["W"], cv["C"]], 70 + i, 1, device=dev) for i in range(4)]
    dY = [inputs.normal([cv["N"], 56, 56, cv["K"]], 70 + i, 3, device=dev) for i in range(4)]
    Wf = inputs.normal([cv["K"], cv["R"], cv["S"], cv["C"]], 70, 2, 1 / 48., device=dev)
    dX = [torch.empty(cv["N"], cv["H"], cv["W"], cv["C"], dtype=bf, device=dev) for _ in range(4)]
    dW = torch.empty(cv["K"], cv["R"], cv["S"], cv["C"], dtype=torch.float32, device=dev)
    timed("conv2d_dgrad_32x56x56x256_k256_3x3", [(lambda i=i: sg.conv2d_dgrad(dY[i], Wf, (56, 56), pad=(1, 1), out=dX[i])) for i in range(4)],
          dict(op="conv2d_dgrad", conv=geo))
    timed("conv2d_wgrad_32x56x56x256_k256_3x3_fp32_dW",
          [(lambda i=i: sg.conv2d_wgrad(dY[i], X[i], (3, 3), pad=(1, 1), out=dW)) for i in range(4)],
          dict(op="conv2d_wgrad", conv=geo, elem_bytes_out=4))
    # a strided layer: 32x56x56x256 -> 512 filters 3x3 stride 2 (output 28x28)
    geo2 = dict(N=32, H=56, W=56, C=256, K=512, R=3, S=3, pad=(1, 1), stride=(2, 2))
    dY2 = [inputs.normal([32, 28, 28, 512], 80 + i, 3, device=dev) for i in range(4)]
    Wf2 = inputs.normal([512, 3, 3, 256], 80, 2, 1 / 48., device=dev)
    dW2 = torch.empty(512, 3, 3, 256, dtype=torch.float32, device=dev)
    timed("conv2d_dgrad_32x56x56x256_k512_3x3_stride2",
          [(lambda i=i: sg.conv2d_dgrad(dY2[i], Wf2, (56, 56), pad=(1, 1), stride=(2, 2), out=dX[i])) for i in range(4)],
          dict(op="conv2d_dgrad", conv=geo2), note="four output phases in one launch")
    timed("conv2d_wgrad_32x56x56x256_k512_3x3_stride2_fp32_dW",
          [(lambda i=i: sg.conv2d_wgrad(dY2[i], X[i], (3, 3), pad=(1, 1), stride=(2, 2), out=dW2)) for i in range(4)],
          dict(op="conv2d_wgrad", conv=geo2, elem_bytes_out=4))
    return out


def profile_config(args) -> None:
    """A few kernel-only launches of one of the configurations c3, c4, c5 inside a cudaProfilerStart/Stop bracket, so that
    `ncu --profile-from-start off` captures that configuration's kernel alone (the default run profiles c2)."""
    import torch
    from paper_2603_29010_b200 import inputs, solgemm as sg
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    C = inputs.CONFIGS
    name = {"c3": "c3_batched_128x256x256x512_gelu", "c4": "c4_conv_32x56x56x256_k256_3x3_bias_relu",
            "c5": "c5_grouped_16xMx4096x4096_silu", "gemv1": "matrix_vector_8192x8192_1_vector",
            "gemv8": "matrix_vector_8192x8192_8_vectors", "transpose": "transpose_8x4096x4096_bf16_to_bf16",
            "splitk": "gemm_256x256x32768_two_pass_split_k"}[args.profile_config]
    c = C.get(name)
    if args.profile_config in ("gemv1", "gemv8"):
        nvec = 1 if args.profile_config == "gemv1" else 8
        sets = 3
        Ws = [torch.randn(8192, 8192, device=dev).to(torch.bfloat16) for _ in range(sets)]
        x = torch.randn(nvec, 8192, device=dev).to(torch.bfloat16)
        outs = [torch.empty(8192, nvec, dtype=torch.bfloat16, device=dev) for _ in range(sets)]
        step = lambda i: sg.gemm(Ws[i % sets], x, out=outs[i % sets])
    elif args.profile_config == "transpose":
        sets = 3
        xs = [torch.randn(8, 4096, 4096, device=dev).to(torch.bfloat16) for _ in range(sets)]
        ys = [torch.empty(8, 4096, 4096, dtype=torch.bfloat16, device=dev) for _ in range(sets)]
        step = lambda i: sg.transpose(xs[i % sets], out=ys[i % sets])
    elif args.profile_config == "splitk":
        sets = 8
        As = [torch.randn(256, 32768, device=dev).to(torch.bfloat16) for _ in range(sets)]
        Bs = [torch.randn(256, 32768, device=dev).to(torch.bfloat16) for _ in range(sets)]
        outs = [torch.empty(256, 256, dtype=torch.bfloat16, device=dev) for _ in range(sets)]
        step = lambda i: sg.gemm(As[i % sets], Bs[i % sets], out=outs[i % sets])
    elif args.profile_config == "c3":
        sets = 4
        data = [inputs.make_gemm(c["M"], c["N"], c["K"], c["dist"], c["scale"], seed=i, device=dev, batch=c["batch"]) for i in range(sets)]
        outs = [torch.empty(c["batch"], c["M"], c["N"], dtype=torch.bfloat16, device=dev) for _ in range(sets)]
        step = lambda i: sg.batched_gemm(data[i % sets][0], data[i % sets][1], out=outs[i % sets], epi=c["epi"])
    elif args.profile_config == "c4":
        sets = 4
        data = [inputs.make_conv(c["N"], c["H"], c["W"], c["C"], c["K"], c["R"], c["S"], c["dist"], c["scale"], bias=True, seed=i,
                                 device=dev) for i in range(sets)]
        outs = [torch.empty(c["N"], 56, 56, c["K"], dtype=torch.bfloat16, device=dev) for _ in range(sets)]
        step = lambda i: sg.conv2d_fprop(data[i % sets][0], data[i % sets][1], pad=c["pad"], bias=data[i % sets][2],
                                         out=outs[i % sets], epi=c["epi"])
    else:
        Ms = inputs.grouped_sizes(c["groups"], c["M_lo"], c["M_hi"])
        As, Bs = inputs.make_grouped(Ms, c["N"], c["K"], c["dist"], c["scale"], device=dev)
        outs = [torch.empty(m, c["N"], dtype=torch.bfloat16, device=dev) for m in Ms]
        ws = torch.empty(sg.grouped_workspace_size(len(Ms)), dtype=torch.uint8, device=dev)
        step = lambda i: sg.grouped_gemm(As, Bs, outs=outs, epi=c["epi"], workspace=ws)
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)      # larger than L2: every timed launch starts cold
    for i in range(max(args.warmup, 3)):
        step(i)
    torch.cuda.synchronize()
    times = []
    torch.cuda.profiler.start()
    for i in range(args.steps):
        flush.zero_()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        step(i)
        e1.record()
        e1.synchronize()
        times.append(e0.elapsed_time(e1) * 1e3)
    torch.cuda.profiler.stop()
    sg.poll_status()
    print(json.dumps({"profile_config": name, "launches": args.steps, "us_per_launch_single_cold": times,
                      "plan": sg.last_launch_plan(), "kernel": sg.last_kernel_name()}), flush=True)


def spread_rows(M: int, count: int, tile_m: int = 256):
    """`count` distinct rows spread over the whole matrix: the first and last row of every tile row, then seeded rows."""
    from paper_2603_29010_b200 import inputs
    rows = []
    for t in range(-(-M // tile_m)):
        rows += [t * tile_m, min(M, (t + 1) * tile_m) - 1]
    rows = sorted(set(rows))[:count]
    seen = set(rows)
    for r in inputs.integers(4 * count, 4242, 14, 0, M - 1):
        if len(rows) >= count:
            break
        if r not in seen:
            seen.add(r)
            rows.append(r)
    return sorted(rows)


def run_ours(args, rank: int, world: int, local_rank: int) -> None:
    import torch
    import torch.distributed as dist
    from paper_2603_29010_b200 import inputs, sharding
    from paper_2603_29010_b200 import solgemm as sg      # raises if the CUDA library is missing

    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device (there is no CPU path)")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    c = inputs.CONFIGS[WORKLOAD]
    M, N, K = c["M"], c["N"], c["K"]
    peaks, peaks_kind = measured_peaks()
    footprint = 2 * (M * K + N * K + M * N) + 2 * N
    sets = -(-4 * L2_BYTES // footprint) + 1                       # distinct buffer sets cycled through: > 4x L2 in total
    data = [inputs.make_gemm(M, N, K, c["dist"], c["scale"], bias=True, seed=inputs.BASE_SEED + 17 * rank + i, device=dev)
            for i in range(sets)]
    outs = [torch.empty(M, N, dtype=torch.bfloat16, device=dev) for _ in range(sets)]

    def step(i):
        A, B, bias = data[i % sets]
        sg.gemm(A, B, bias=bias, out=outs[i % sets], epi=c["epi"])

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def max_over_ranks(x: float) -> float:
        if world == 1:
            return x
        t = torch.tensor([x], dtype=torch.float64, device=dev)
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return float(t.item())

    for i in range(max(args.warmup, 3)):
        step(i)
    barrier()
    sampler = ClockSampler(physical_gpu_index(local_rank))
    sampler.start()
    # The K timed steps are one CUDA graph (K kernel nodes, one per step, each on the next buffer set), replayed once
    # untimed (the upload) and once timed; the same K steps as plain launches are timed first and reported beside it.
    dt_plain = time_steps(step, args.steps, torch)
    barrier()
    launches0 = sg.launch_count()
    timed_graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(timed_graph):
        for i in range(args.steps):
            step(i)
    launches = sg.launch_count() - launches0      # kernel nodes of the graph = launches of the timed region
    plan = sg.last_launch_plan()                 # of the timed launches (read before anything else is launched)
    kernel_name = sg.last_kernel_name()
    timed_graph.replay()
    barrier()
    torch.cuda.profiler.start()            # lets `ncu --profile-from-start off` see the timed region only
    dt = time_steps(lambda i: timed_graph.replay(), 1, torch)
    torch.cuda.profiler.stop()
    sampler.sample_once()
    kernel_mhz = sg.last_kernel_clock_mhz()      # cycle counter / ns timer inside the last timed kernel
    barrier()
    clocks = sampler.stop()
    clocks["sm_mhz_in_kernel"] = round(kernel_mhz, 1)
    clocks["note"] = "sm_mhz is the management library's figure (on this pool: the requested clock); sm_mhz_in_kernel is counted inside the timed kernel"
    sg.poll_status()
    dt = max_over_ranks(dt)
    dt_plain = max_over_ranks(dt_plain)

    # ---- burst and sustained, side by side (one GPU's figure; every rank runs it so that the GPUs stay in step)
    burst, sustained_rec = None, None
    if not args.kernel_only:
        import time as _time
        fns = [(lambda i=i: step(i)) for i in range(sets)]
        graph = torch.cuda.CUDAGraph()
        torch.cuda.synchronize()
        with torch.cuda.graph(graph):
            for f in fns:
                f()
        b_times, b_mhz = [], []
        for _ in range(5):
            torch.cuda.synchronize()
            _time.sleep(0.25)                    # let the board settle: a burst starts from an idle GPU
            graph.replay()                       # one untimed pass to wake the clocks, then 2 x `sets` timed launches
            b_times.append(time_steps(lambda i: graph.replay(), 2, torch) / (2 * sets))
            b_mhz.append(sg.last_kernel_clock_mhz())
        n_sus = max(8, int(0.6 / (min(b_times) * sets)))      # at least 0.6 s of back-to-back launches
        t_sus = time_steps(lambda i: graph.replay(), n_sus, torch) / (n_sus * sets)
        sus_mhz = sg.last_kernel_clock_mhz()
        flops2 = 2.0 * M * N * K
        burst = {"us_median": _median(b_times) * 1e6, "us_best": min(b_times) * 1e6, "repeats": len(b_times),
                 "launches_per_repeat": 2 * sets, "tflops_median": flops2 / _median(b_times) / 1e12,
                 "frac_of_burst_peak": flops2 / _median(b_times) / 1e12 / peaks["bf16_tflops"],
                 "sm_mhz_in_kernel": round(_median(b_mhz), 1)}
        sustained_rec = {"us": t_sus * 1e6, "seconds": t_sus * n_sus * sets, "tflops": flops2 / t_sus / 1e12,
                         "frac_of_sustained_peak": flops2 / t_sus / 1e12 / peaks["bf16_tflops_sustained"],
                         "sm_mhz_in_kernel": round(sus_mhz, 1),
                         "tflops_per_ghz": flops2 / t_sus / 1e12 / (sus_mhz / 1e3) if sus_mhz else None}
        del graph
        barrier()

    # ---- end to end: pinned host buffers, copies inside the timed region
    e2e_steps = max(3, min(args.steps, 20))
    dt_e2e = float("nan")
    if not args.kernel_only:
        hA, hB, hb = (t.cpu().pin_memory() for t in data[0])
        hD = torch.empty(M, N, dtype=torch.bfloat16).pin_memory()
        scratch = {}
        for _ in range(3):
            sg.gemm_host(hA, hB, hD, bias_host=hb, epi=c["epi"], device=dev, scratch=scratch)
        barrier()
        dt_e2e = time_steps(lambda i: sg.gemm_host(hA, hB, hD, bias_host=hb, epi=c["epi"], device=dev, scratch=scratch),
                            e2e_steps, torch)
        barrier()
        dt_e2e = max_over_ranks(dt_e2e)
        del scratch
    h2d = 2 * (M * K + N * K) + 2 * N
    d2h = 2 * M * N

    flops = 2.0 * M * N * K
    per_launch = dt / args.steps
    achieved = flops / per_launch / 1e12
    # Denominator: the burst cuBLAS figure for short timed regions; the sustained one when the region ran long
    # enough (>= 0.1 s of back-to-back launches) to be held at the board's power cap.  Evidence of the cap: the
    # driver's sw_power_cap reason, or (the management library on this pool reports the requested clock and no reason)
    # the SM clock counted inside the kernel sitting below three quarters of the maximum.
    in_kernel = clocks.get("sm_mhz_in_kernel") or 0.0
    capped = "sw_power_cap" in clocks["reasons"] or (0.0 < in_kernel < 0.75 * float(clocks.get("sm_max_mhz") or 1965))
    sustained = dt >= 0.1 and capped
    peak = peaks["bf16_tflops_sustained"] if sustained else peaks["bf16_tflops"]
    sol_spec = sg.sol_bound("gemm", M=M, N=N, K=K, has_bias=1, peak_flops=SPEC_PEAK_FLOPS, peak_bytes_per_s=SPEC_PEAK_BW)
    sol_meas = sg.sol_bound("gemm", M=M, N=N, K=K, has_bias=1, peak_flops=peaks["bf16_tflops"] * 1e12,
                            peak_bytes_per_s=peaks["hbm_gbs"] * 1e9)
    # the paper's clock rule (Section 4.1): datasheet peak x current / maximum clock
    sol_clock = sg.sol_bound("gemm", M=M, N=N, K=K, has_bias=1, peak_flops=SPEC_PEAK_FLOPS, peak_bytes_per_s=SPEC_PEAK_BW,
                             sm_clock_mhz=float(kernel_mhz or clocks["sm_mhz"] or 0),
                             sm_clock_max_mhz=float(clocks["sm_max_mhz"] or 0))
    # the same rule on the per-clock capability of the tensor pipes (8192 FLOP per SM clock x 148 SMs)
    per_clock_peak = PER_CLOCK_FLOPS * float(kernel_mhz or 0) * 1e6

    # ---- every configuration, this rank's shard of each (N = 1: the whole problems), max over ranks
    per_config = None
    if not args.kernel_only:
        del data[1:], outs[1:]
        torch.cuda.empty_cache()
        per_config = bench_per_config(sg, inputs, sharding, torch, dist, dev, peaks, rank, world, torch_ref=not args.no_torch_ref)
        sg.poll_status()

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    line = {
        "metric": METRIC, "value": world * achieved, "unit": "TFLOP/s", "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": per_launch * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
        "config": {"workload": WORKLOAD, "M": M, "N": N, "K": K, "layout": "A row-major, B column-major",
                   "epilogue": "bias+relu", "accumulate": "fp32", "out": "bf16",
                   "l2": f"inputs larger than L2: {sets} distinct buffer sets ({sets * footprint / 1e6:.0f} MB) used in turn",
                   "launch": "the K timed steps are the K kernel nodes of one CUDA graph (replayed once untimed, once timed, CUDA "
                             "events around the timed replay); ms_per_step_plain_launches is the same K steps as plain launches",
                   "per_gpu": "value: every rank runs the whole problem on its own GPU (no collective); per_config: every "
                              "rank runs its shard of each problem (rows / batch entries / images / whole groups)"},
        "clocks": clocks,
        "e2e": {"value": world * flops / (dt_e2e / e2e_steps) / 1e12, "unit": "TFLOP/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": d2h, "steps": e2e_steps, "ms_per_step": dt_e2e / e2e_steps * 1e3},
        "ms_per_step_plain_launches": dt_plain / args.steps * 1e3,
        "gpu_launches": launches,
        "kernels_in_timed_region": {
            "names": [kernel_name], "launches": launches, "one_launch_per_step": bool(launches == args.steps),
            "library_kernel_names_present": bool(__import__("re").search(r"cublas|cutlass|cudnn|at::native", kernel_name)),
            "source": "the library's own launch record (sg_last_kernel_name, sg_launch_count): the timed region calls "
                      "sg_gemm only, which launches exactly this one kernel per step"},
        "roofline": {"bound": "tensor", "achieved": achieved, "peak": peak, "unit": "TFLOP/s", "frac": achieved / peak,
                     "traffic": NCU_DRAM_BYTES_PER_LAUNCH, "traffic_source": NCU_DRAM_SOURCE,
                     "algorithmic_flops_per_launch": int(flops),
                     "algorithmic_bytes_per_launch": int(sol_spec["bytes"]),
                     "peak_source": f"{'sustained' if sustained else 'burst'} cuBLAS bf16 of {peaks_kind} peaks",
                     "frac_of_burst_peak": achieved / peaks["bf16_tflops"],
                     "frac_of_sustained_peak": achieved / peaks["bf16_tflops_sustained"],
                     "per_clock_tensor_peak": per_clock_peak / 1e12 if per_clock_peak else None,
                     "frac_of_per_clock_tensor_peak": achieved * 1e12 / per_clock_peak if per_clock_peak else None,
                     "tiling": plan, "kernel": kernel_name},
        "sol": {"flops": sol_spec["flops"], "bytes": sol_spec["bytes"], "ai": sol_spec["ai"],
                "t_sol_us_spec": sol_spec["t_sol_s"] * 1e6, "frac_of_sol_spec": sol_spec["t_sol_s"] / per_launch,
                "t_sol_us_measured_peaks": sol_meas["t_sol_s"] * 1e6, "frac_of_sol_measured_peaks": sol_meas["t_sol_s"] / per_launch,
                "t_sol_us_clock_scaled": sol_clock["t_sol_s"] * 1e6, "frac_of_sol_clock_scaled": sol_clock["t_sol_s"] / per_launch,
                "clock_scaled_rule": "datasheet peak x in-kernel SM clock / maximum SM clock",
                "suspicious_faster_than_0.9_sol": bool(per_launch < 0.9 * sol_spec["t_sol_s"])},
    }
    if burst is not None:
        line["c2_burst"], line["c2_sustained"] = burst, sustained_rec
    if per_config is not None:
        line["per_config"] = per_config

    if args.kernel_only:
        line["e2e"] = None
    if world == 1 and not args.kernel_only:
        from oracle import oracle as orc
        hA2, hB2, hb2 = (t.cpu() for t in data[0])
        nrows, _ = oracle_rows_for(12.0, hA2, hB2, hb2, c["epi"], M)
        rows = spread_rows(M, nrows)
        idx = torch.tensor(rows)
        subA = hA2[idx].contiguous()
        t0 = time.perf_counter()
        ref, absacc = orc.gemm(subA, hB2, bias=hb2, epi=c["epi"])
        cpu_dt = time.perf_counter() - t0
        line["cpu_baseline"] = {"value": 2.0 * len(rows) * N * K / cpu_dt / 1e12, "unit": "TFLOP/s", "cores": orc.num_threads(),
                                "kind": "oracle", "seconds": cpu_dt,
                                "sample": f"{len(rows)} of {M} output rows spread over the matrix (first and last row of every "
                                          f"256-row tile, then seeded rows; {len(rows) * N} of {M * N} elements), all N and K"}
        # the same rows double as a parity spot check of the timed configuration
        step(0)
        torch.cuda.synchronize()
        got = outs[0][idx.to(dev)].cpu().double()
        line["parity_sample_ok"] = bool(((got - ref).abs() <= 1e-2 + 1e-2 * ref.abs()).all())
        if args.widened:
            line["widened"] = bench_widened(sg, inputs, torch, dev, peaks)
        if args.shape_sweep:
            line["shape_sweep"] = bench_shape_sweep(sg, torch, dev)
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=2000)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--no-torch-ref", action="store_true", help="skip the torch library reference timings in per_config")
    ap.add_argument("--shape-sweep", action="store_true",
                    help="also time the workload list's GEMM shape classes, with torch's library kernels beside them")
    ap.add_argument("--widened", action="store_true",
                    help="also time the rows built beyond the five configurations (epilogue chain, dtypes, layouts, "
                         "skinny shapes, transpose, conv gradients; N=1 only)")
    ap.add_argument("--profile-config", choices=["c3", "c4", "c5", "gemv1", "gemv8", "transpose", "splitk"], default=None,
                    help="only run a few launches of that configuration inside the profiler bracket (for ncu)")
    ap.add_argument("--kernel-only", action="store_true",
                    help="skip the end-to-end and CPU-baseline legs (for profiler captures of the timed kernel)")
    args = ap.parse_args()

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if args.gpus > 1 and world == 1:
        # not under torchrun: start one process per GPU on this node
        port = os.environ.get("MASTER_PORT", "29511")
        cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
               "--master-addr", "127.0.0.1", "--master-port", port, os.path.abspath(__file__)] + sys.argv[1:]
        sys.exit(subprocess.call(cmd))
    if args.profile_config:
        if world > 1 or args.impl != "ours":
            raise SystemExit("--profile-config is a single-GPU mode of the CUDA arm")
        profile_config(args)
        return
    if args.impl == "reference":
        if args.steps < 1:
            args.steps = 1
        run_reference(args, rank, world)
    else:
        run_ours(args, rank, world, local_rank)


if __name__ == "__main__":
    main()
