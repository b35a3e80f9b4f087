#!/usr/bin/env python
"""Benchmark of the SC-GEMM hot path on B200.

A step is one pass of the whole path over one batch: row metric (sc_row_stats) -> stream-length
assignment (sc_assign_lengths) -> sc_matmul (scales, row ordering, encode of A and W, bit-serial GEMM
core, decode).  Default workload: the ViT-B/16 MLP fc1 shape, A[1576 x 768] x W[768 x 3072], bipolar
XNOR, uniform L = 128.  Metric: stream bit-ops/s = N * K * sum_i L_i / t (Sec. 4.1 cost model), with the
equivalent MAC/s beside it.

    python bench.py --gpus N --steps K --warmup W          (N > 1: launched by torch.distributed.run)
    python bench.py --impl reference ...                    times the CPU oracle on a bounded sample

Prints ONE JSON line (rank 0).
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "sc_gemm_stream_bitops_per_s"
UNIT = "bitop/s"
MODES = {"bipolar": 0, "unipolar": 1}
SCALES = {"none": 0, "per_row": 1, "per_tensor": 2}
L2_FLUSH_BYTES = 256 << 20

# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of one core-kernel launch, from an
# `ncu --set full` capture of this command on the workload named by the key.
NCU_CORE_TRAFFIC_BYTES = {("vit_b16_fc1", "alu"): 85.4e6, ("vit_b16_fc1", "umma"): 93.8e6, ("vit_b16_fc1", "pair"): 93.9e6,
                          ("vit_l14_fc1_L128", "pair"): 7.21e9}

FP4_TO_BF16_NOMINAL = 4.0       # dense tensor peaks: 9 PFLOP/s fp4 vs 2.25 PFLOP/s bf16

# Integer-pipe ceiling of the plain gate+popcount core: POPC issues at 16 lanes/clk/SM, each POPC
# retires 32 stream bit-ops; 148 SMs at the maximum SM clock.
POPC_PER_CLK_PER_SM = 16

# Beside the headline workload the default run times these for a few steps each (kernels launched one by one): the
# per-row mixed-precision configuration, the grouped DiT-like one, and the widest bipolar and the unipolar layer of the
# ViT-L/14 sweep at L = 128.
OTHER_CONFIGS = ("vit_b16_qkv_mixed", "dit_xl2_linear_grouped", "vit_l14_fc1_L128", "vit_l14_fc2_L128")


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", choices=["ours", "reference"], default="ours")
    ap.add_argument("--config", default="vit_b16_fc1", help="workload name (see workloads.all_configs)")
    ap.add_argument("--core", type=int, default=0, help="GEMM core variant (0 auto, 1 popc, 2 carry-save, 3 simple, 4 one-SM tensor core, "
                    "5 two-SM tensor core)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-graph", action="store_true", help="launch the step's kernels one by one instead of replaying "
                                                            "a CUDA graph captured from the same calls")
    ap.add_argument("--microbench", action="store_true", help="also report measured integer-pipe peaks")
    ap.add_argument("--no-configs", action="store_true", help="skip the short runs of the other benchmark configurations")
    ap.add_argument("--sweep", metavar="FILE", help="time every benchmark configuration (all five configs, every "
                    "L of the ViT-L sweep) and write a table to FILE instead of the JSON line")
    ap.add_argument("--attention", metavar="FILE", help="time the batched attention products (qk and av per head, "
                                                        "ViT-B/16 and ViT-L/14 shapes) and write a markdown table to FILE")
    ap.add_argument("--cbsg", metavar="FILE", help="time the Sobol-8 / conditional-generation product (sc_matmul_cbsg) "
                                                   "on the linear-layer shapes and write a markdown table to FILE")
    return ap.parse_args()


def get_workload(name):
    from paper_2609_32922_b200 import workloads as wl
    cfgs = wl.all_configs()
    if name not in cfgs:
        raise SystemExit("unknown config %r; choose from %s" % (name, ", ".join(sorted(cfgs))))
    return cfgs[name]


class ClockSampler:
    """Samples SM clocks and throttle reasons (read-only NVML queries) every few milliseconds in a thread
    while the timed region runs; falls back to polling nvidia-smi when NVML cannot be loaded."""
    SLOWDOWN_BITS = {0x8: "hw_slowdown", 0x40: "hw_thermal_slowdown", 0x20: "sw_thermal_slowdown", 0x4: "sw_power_cap"}

    def __init__(self, gpu_index):
        self.gpu_index = gpu_index
        self.samples, self.reasons, self.max_mhz = [], set(), None
        self._stop = threading.Event()
        self._first = threading.Event()          # set once the first sample has landed (or sampling is impossible)
        self._thread = None

    def _physical_index(self):
        vis = os.environ.get("CUDA_VISIBLE_DEVICES")
        if vis:
            try:
                return int(vis.split(",")[self.gpu_index])
            except (ValueError, IndexError):
                pass
        return self.gpu_index

    def _run_nvml(self):
        import pynvml
        pynvml.nvmlInit()
        h = pynvml.nvmlDeviceGetHandleByIndex(self._physical_index())
        self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        while not self._stop.is_set():
            self.samples.append(float(pynvml.nvmlDeviceGetClockInfo(h, pynvml.NVML_CLOCK_SM)))
            self._first.set()
            try:
                bits = pynvml.nvmlDeviceGetCurrentClocksEventReasons(h)
            except Exception:
                bits = pynvml.nvmlDeviceGetCurrentClocksThrottleReasons(h)
            for bit, name in self.SLOWDOWN_BITS.items():
                if bits & bit:
                    self.reasons.add(name)
            time.sleep(0.003)
        pynvml.nvmlShutdown()

    def _run_smi(self):
        q = "clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown," \
            "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap"
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        while not self._stop.is_set():
            try:
                out = subprocess.run(["nvidia-smi", "-i", str(self._physical_index()), "--query-gpu=" + q,
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
                f = [x.strip() for x in out.strip().split(",")]
                self.samples.append(float(f[0]))
                self.max_mhz = float(f[1])
                self._first.set()
                for name, val in zip(names, f[2:6]):
                    if val.lower().startswith("active"):
                        self.reasons.add(name)
            except Exception:
                self._first.set()
                return

    def _run(self):
        try:
            self._run_nvml()
        except Exception:
            self._run_smi()
        self._first.set()

    def start(self):
        self._thread = threading.Thread(target=self._run, daemon=True)
        self._thread.start()
        # The first sample must land before the timed region starts: loading NVML in a cold process can take longer than a
        # short timed region lasts, which would leave the run without a clock record.
        self._first.wait(timeout=20.0)

    def stop(self):
        self._stop.set()
        if self._thread is not None:
            self._thread.join(timeout=15)
        out = {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}
        if self.samples:
            out["sm_mhz"] = statistics.median(self.samples)
        return out


def measured_peaks():
    try:
        return json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))
    except (OSError, ValueError):
        return {}


def oracle_sample(w, n_rows, n_cols):
    """Times the CPU oracle, as it stands, on n_rows x n_cols output entries of workload w."""
    import numpy as np
    from oracle import sc_oracle
    from paper_2609_32922_b200 import workloads as wl
    sc_oracle.build()
    A, W = wl.make_inputs(w)
    if w.policy:
        avg, Lmin, Lmax, group = w.policy
        Lg, _ = sc_oracle.assign_lengths(sc_oracle.row_absmax(A), group, avg, Lmin, Lmax)
        L_rows = sc_oracle.expand_lengths(Lg, w.M, group)
    else:
        L_rows = np.full(w.M, w.uniform_L, np.int32)
    rows, cols = wl.sample_rows_cols(w, L_rows, n_rows, n_cols)

    def run():
        t0 = time.perf_counter()
        sc_oracle.matmul(A, W, L_rows, MODES[w.mode], SCALES[w.scale_a], SCALES[w.scale_w], w.seed, w.stream_id,
                         row_sel=rows, col_sel=cols)
        return time.perf_counter() - t0

    bitops = float(len(cols)) * w.K * float(L_rows[rows].sum())
    sample = "%d rows x %d columns of %s (all K, full stream lengths), scales over the full tensors" % (
        len(rows), len(cols), w.name)
    return run, bitops, sample, sc_oracle.num_threads()


def run_reference(args):
    """The oracle as the reference arm: each step is a bounded sample of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = get_workload(args.config)
    run, bitops, sample, cores = oracle_sample(w, 32, 256)
    for _ in range(args.warmup):
        run()
    times = [run() for _ in range(args.steps)]
    total = sum(times)
    value = bitops * args.steps / total
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "u8 stream bits / int32 counts",
        "data": "synthetic", "config": {"workload": w.name, "M": w.M, "K": w.K, "N": w.N, "mode": w.mode,
                                         "L": w.uniform_L if w.uniform_L else "policy", "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "equiv_mac_per_s": value / (w.uniform_L if w.uniform_L else w.policy[0]),
        "gpu_launches": 0,
    }
    print(json.dumps(line))


def measure_workload(sc, dev, name, core, reps=None):
    """One workload through the public calls, kernels launched one by one: the whole step (min of `reps` runs, CUDA events
    on the launching stream), the core phase from the library's own phase events, and the same step with prepared weights.
    Operands of every workload here exceed the L2 capacity together with their stream planes, or are flushed by the
    next workload's allocation; the headline line of the default run flushes L2 explicitly instead."""
    import torch
    from paper_2609_32922_b200 import binding, workloads as wl
    w = get_workload(name)
    A_h, W_h = wl.make_inputs(w)
    A, W = torch.from_numpy(A_h).to(dev), torch.from_numpy(W_h).to(dev)
    if w.policy:
        avg, Lmin, Lmax, group = w.policy
    else:
        avg, Lmin, Lmax, group = float(w.uniform_L), min(8, w.uniform_L), w.uniform_L, 1
    params = binding.make_params(mode=MODES[w.mode], scale_a=SCALES[w.scale_a], scale_w=SCALES[w.scale_w],
                                 group=group, seed=w.seed, core=core)
    g = torch.empty(w.M, dtype=torch.float32, device=dev)
    L = torch.empty((w.M + group - 1) // group, dtype=torch.int32, device=dev)
    C = torch.empty((w.M, w.N), dtype=torch.float32, device=dev)
    ws = sc.workspace(binding.sc_workspace_bytes(w.M, w.K, w.N, Lmax, params))
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)

    def step():
        binding.sc_row_stats(sc.ctx, A, g)
        binding.sc_assign_lengths(sc.ctx, g, group, avg, Lmin, Lmax, L)
        binding.sc_matmul(sc.ctx, A, W, L, Lmax, params, None, C, ws)

    if reps is None:
        reps = 3 if w.M * w.N * w.K * Lmax < 2e13 else 1
    for _ in range(2 if reps > 1 else 1):
        step()
    torch.cuda.synchronize()
    binding.sc_profile_enable(sc.ctx, True)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    step_ms, core_ms = [], []
    for _ in range(reps):
        flush.zero_()
        e0.record()
        step()
        e1.record()
        torch.cuda.synchronize()
        step_ms.append(e0.elapsed_time(e1))
        core_ms.append(binding.sc_profile_read(sc.ctx)["core"])
    binding.sc_profile_enable(sc.ctx, False)
    # the same step with the W side prepared once (static weights)
    prepared = sc.prepare_weights(W, Lmax, params)

    def step_prepared():
        binding.sc_row_stats(sc.ctx, A, g)
        binding.sc_assign_lengths(sc.ctx, g, group, avg, Lmin, Lmax, L)
        binding.sc_matmul_prepared(sc.ctx, A, prepared[0], L, Lmax, params, None, C, ws)

    step_prepared()
    prep_ms = []
    for _ in range(reps):
        flush.zero_()
        e0.record()
        step_prepared()
        e1.record()
        torch.cuda.synchronize()
        prep_ms.append(e0.elapsed_time(e1))
    binding.sc_weights_release(prepared[0])
    sum_L = float(oracle_free_sum_lengths(L, group, w.M))
    bitops = float(w.N) * w.K * sum_L
    out = {"workload": name, "M": w.M, "K": w.K, "N": w.N, "mode": w.mode, "mean_L": sum_L / w.M, "bitops": bitops,
           "step_ms": min(step_ms), "core_ms": min(core_ms), "prepared_step_ms": min(prep_ms), "reps": reps,
           "tensor_core": core in (0, 4) and w.K * Lmax <= (1 << 24)}
    del A, W, C, prepared, ws, flush
    return out


def run_sweep(args):
    """Every configuration once: whole-step and core-only throughput, written as a markdown table."""
    import torch
    from paper_2609_32922_b200 import binding, build, workloads as wl
    build.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    sc = binding.ScGemm(0)
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    sm_max = float(measured_peaks().get("sm_max_mhz") or 1965.0)
    alu_peak = POPC_PER_CLK_PER_SM * 32.0 * n_sm * sm_max * 1e6
    names = ["tiny_bipolar", "vit_b16_fc1", "vit_b16_qkv_mixed", "dit_xl2_linear_grouped"]
    for L in wl.VIT_L_SWEEP_L:
        names += [w.name for w in wl.vit_l_layers(L)]
    rows = []
    for name in names:
        m = measure_workload(sc, dev, name, args.core)
        t, tc, tp, bitops = m["step_ms"] * 1e-3, m["core_ms"] * 1e-3, m["prepared_step_ms"] * 1e-3, m["bitops"]
        rows.append((name, m["M"], m["K"], m["N"], m["mode"], m["mean_L"], bitops, t * 1e3, bitops / t,
                     float(m["M"]) * m["N"] * m["K"] / t, tc * 1e3, bitops / tc, bitops / tc / alu_peak, tp * 1e3,
                     bitops / tp))
    assert sc.device_status() == 0
    with open(args.sweep, "w") as f:
        f.write("| workload | M | K | N | mode | mean L | bit-ops | step ms | step bit-op/s | equiv MAC/s | core ms | "
                "core bit-op/s | core / POPC bound | step ms, W prepared | bit-op/s, W prepared |\n"
                "|---|---|---|---|---|---|---|---|---|---|---|---|---|---|---|\n")
        for r in rows:
            f.write("| %s | %d | %d | %d | %s | %.1f | %.3g | %.3f | %.3g | %.3g | %.3f | %.3g | %.2f | %.3f | %.3g |\n" % r)
    print("wrote", args.sweep, file=sys.stderr)


def run_attention(args):
    """Batched attention products through sc_matmul_batched: whole-step and core times per workload."""
    import torch
    from paper_2609_32922_b200 import binding, build, workloads as wl
    build.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    sc = binding.ScGemm(0)
    rows = []
    for w in wl.attention_workloads(128) + wl.attention_workloads(32):
        A_h, W_h, transposed = wl.make_attention_inputs(w)
        B, M, K, N = w.shape
        A, W = torch.from_numpy(A_h).to(dev), torch.from_numpy(W_h).to(dev)
        params = binding.make_params(mode=MODES[w.mode], scale_a=SCALES["per_row"], scale_w=SCALES["per_tensor"],
                                     seed=w.seed, core=args.core)
        g = torch.empty(B * M, dtype=torch.float32, device=dev)
        L = torch.empty(B * M, dtype=torch.int32, device=dev)
        C = torch.empty((B, M, N), dtype=torch.float32, device=dev)
        ws = sc.workspace(binding.sc_workspace_bytes_batched(B, M, K, N, w.L, params))

        def step():
            binding.sc_row_stats(sc.ctx, A.view(B * M, K), g)
            binding.sc_assign_lengths(sc.ctx, g, 1, float(w.L), min(8, w.L), w.L, L)
            binding.sc_matmul_batched(sc.ctx, A, W, transposed, L, w.L, params, None, C, ws)

        for _ in range(2):
            step()
        torch.cuda.synchronize()
        binding.sc_profile_enable(sc.ctx, True)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        step_ms, core_ms = [], []
        for _ in range(3):
            e0.record()
            step()
            e1.record()
            torch.cuda.synchronize()
            step_ms.append(e0.elapsed_time(e1))
            core_ms.append(binding.sc_profile_read(sc.ctx)["core"])
        binding.sc_profile_enable(sc.ctx, False)
        bitops = float(B) * M * N * K * w.L
        t, tc = min(step_ms) * 1e-3, min(core_ms) * 1e-3
        tiles = (N + 191) // 192                              # the one-SM tensor-core core spreads N evenly over its tiles,
        tile_n = min(192, round_up((N + tiles - 1) // tiles, 32))   # in multiples of 32 columns
        pad = (round_up(M, 128) * tiles * tile_n) / float(M * N)
        rows.append((w.name, B, M, K, N, w.mode, w.L, bitops, t * 1e3, bitops / t, tc * 1e3, bitops / tc, pad))
        del A, W, C
    assert sc.device_status() == 0
    with open(args.attention, "w") as f:
        f.write("| workload | heads | M | K | N | mode | L | bit-ops | step ms | step bit-op/s | core ms | core bit-op/s | "
                "tile padding (x work) |\n|---|---|---|---|---|---|---|---|---|---|---|---|---|\n")
        for r in rows:
            f.write("| %s | %d | %d | %d | %d | %s | %d | %.3g | %.3f | %.3g | %.3f | %.3g | %.2f |\n" % r)
    print("wrote", args.attention, file=sys.stderr)


def run_cbsg(args):
    """sc_matmul_cbsg on the linear-layer shapes: a row of length L is a code of 2 L positions."""
    import torch
    from paper_2609_32922_b200 import binding, build, workloads as wl
    build.build()
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    sc = binding.ScGemm(0)
    rows = []
    names = ["vit_b16_fc1", "vit_l14_qkv_L128", "vit_l14_proj_L128", "vit_l14_fc1_L128"]
    for name in names:
        w = get_workload(name)
        A_h, W_h = wl.make_inputs(w)
        A, W = torch.from_numpy(A_h).to(dev), torch.from_numpy(W_h).to(dev)
        params = binding.make_params(mode=0, scale_a=SCALES[w.scale_a], scale_w=SCALES[w.scale_w], seed=w.seed)
        C = torch.empty((w.M, w.N), dtype=torch.float32, device=dev)
        ws = sc.workspace(binding.sc_workspace_bytes_cbsg(w.M, w.K, w.N, 256, params))
        for L in (128, 256):
            for _ in range(2):
                binding.sc_matmul_cbsg(sc.ctx, A, W, None, L, params, None, C, ws)
            torch.cuda.synchronize()
            binding.sc_profile_enable(sc.ctx, True)
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            best, phases = None, None
            for _ in range(3):
                e0.record()
                binding.sc_matmul_cbsg(sc.ctx, A, W, None, L, params, None, C, ws)
                e1.record()
                torch.cuda.synchronize()
                ms = e0.elapsed_time(e1)
                if best is None or ms < best:
                    best, phases = ms, binding.sc_profile_read(sc.ctx)
            binding.sc_profile_enable(sc.ctx, False)
            stream_bitops = float(w.M) * w.N * w.K * L
            code_bitops = float(w.M) * w.N * w.K * 2 * L
            rows.append((name.replace("_L128", ""), w.M, w.K, w.N, L, best, stream_bitops / (best * 1e-3), phases["encode_a"],
                         phases["encode_w"], phases["core"], code_bitops / (phases["core"] * 1e-3)))
        del A, W, C
    assert sc.device_status() == 0
    with open(args.cbsg, "w") as f:
        f.write("| shape | M | K | N | L | call ms | stream bit-op/s (N K M L / t) | encode A ms | encode W ms | core ms | "
                "core code bit-op/s (N K M 2L / t) |\n|---|---|---|---|---|---|---|---|---|---|---|\n")
        for r in rows:
            f.write("| %s | %d | %d | %d | %d | %.3f | %.3g | %.3f | %.3f | %.3f | %.3g |\n" % r)
    print("wrote", args.cbsg, file=sys.stderr)


def round_up(x, m):
    return (x + m - 1) // m * m


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.attention:
        run_attention(args)
        return
    if args.cbsg:
        run_cbsg(args)
        return
    if args.sweep:
        run_sweep(args)
        return

    import numpy as np
    import torch
    from paper_2609_32922_b200 import binding, build, dist as scdist, workloads as wl

    rank, world_size, local_rank = scdist.world()
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the SC-GEMM library has no CPU path")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    if world_size > 1:
        scdist.init_process_group("nccl")
    build.build()

    w = get_workload(args.config)
    # weak scaling: every rank owns its own batch of the same shape (different data, same weights)
    import dataclasses
    wr = dataclasses.replace(w, seed=w.seed) if rank == 0 else dataclasses.replace(w, stream_id=rank)
    A_h, W_h = wl.make_inputs(w)
    if rank:
        A_h = np.random.default_rng(w.seed * 1000 + rank).standard_normal(A_h.shape, dtype=np.float32) \
            if w.a_dist.startswith("normal") else A_h
    sc = binding.ScGemm(local_rank)
    params = binding.make_params(mode=MODES[w.mode], scale_a=SCALES[w.scale_a], scale_w=SCALES[w.scale_w],
                                 group=w.group, seed=w.seed, stream_id=wr.stream_id, core=args.core)
    if w.policy:
        avg, Lmin, Lmax, group = w.policy
    else:
        avg, Lmin, Lmax, group = float(w.uniform_L), min(8, w.uniform_L), w.uniform_L, 1

    A = torch.from_numpy(A_h).to(dev)
    W = torch.from_numpy(W_h).to(dev)
    n_groups = (w.M + group - 1) // group
    g = torch.empty(w.M, dtype=torch.float32, device=dev)
    L = torch.empty(n_groups, dtype=torch.int32, device=dev)
    C = torch.empty((w.M, w.N), dtype=torch.float32, device=dev)
    P = torch.empty((w.M, w.N), dtype=torch.int32, device=dev)
    ws = sc.workspace(binding.sc_workspace_bytes(w.M, w.K, w.N, Lmax, params))
    flush = torch.empty(L2_FLUSH_BYTES, dtype=torch.uint8, device=dev)
    stream = torch.cuda.current_stream()

    def step():
        binding.sc_row_stats(sc.ctx, A, g)
        binding.sc_assign_lengths(sc.ctx, g, group, avg, Lmin, Lmax, L)
        binding.sc_matmul(sc.ctx, A, W, L, Lmax, params, P, C, ws)

    def timed_steps(n, fn):
        """n steps, each bracketed by CUDA events on the launching stream, L2 flushed in between."""
        evs = []
        for _ in range(n):
            flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            fn()
            e1.record(stream)
            evs.append((e0, e1))
        torch.cuda.synchronize()
        return [e0.elapsed_time(e1) for e0, e1 in evs]

    # ---- warm-up, then the timed region -------------------------------------------------------------
    for _ in range(max(args.warmup, 3)):
        step()
    torch.cuda.synchronize()
    # The step is a fixed sequence of asynchronous launches on one stream (no host synchronisation inside), so
    # it is captured once into a CUDA graph and replayed: same kernels, same arguments, one launch per step.
    eager_step, graphed = step, False
    if not args.no_graph:
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            eager_step()
        step = graph.replay
        graphed = True
        stream = torch.cuda.current_stream()
        for _ in range(3):
            step()
        torch.cuda.synchronize()
    sum_L = float(oracle_free_sum_lengths(L, group, w.M))
    bitops_per_step = float(w.N) * w.K * sum_L
    launches0 = binding.sc_launch_count(sc.ctx)

    sampler = ClockSampler(local_rank)
    if rank == 0:
        sampler.start()
    scdist.barrier()
    torch.cuda.synchronize()
    times = timed_steps(args.steps, step)
    torch.cuda.synchronize()
    scdist.barrier()
    launches = binding.sc_launch_count(sc.ctx) - launches0
    if graphed:                       # replays do not pass through the library's launch counter
        c0 = binding.sc_launch_count(sc.ctx)
        eager_step()
        torch.cuda.synchronize()
        launches = (binding.sc_launch_count(sc.ctx) - c0) * args.steps
    total_ms = scdist.max_over_ranks(sum(times), dev)
    status = sc.device_status()
    if status != 0:
        raise SystemExit("device status %d (%s) during the timed region" % (status, binding.status_string(status)))

    # ---- per-phase times of the dominant kernel (events recorded by the library around its phases) ----
    binding.sc_profile_enable(sc.ctx, True)
    core_ms, phases = [], []
    for _ in range(min(args.steps, 5)):
        flush.zero_()
        eager_step()
        ph = binding.sc_profile_read(sc.ctx)
        core_ms.append(ph["core"])
        phases.append(ph)
    binding.sc_profile_enable(sc.ctx, False)

    # ---- the same step with prepared weights (static W: its scales, streams and popcount tables built once,
    # outside the timed region).  Reported beside the headline value, never instead of it.
    prepared = sc.prepare_weights(W, Lmax, params)

    def step_prepared():
        binding.sc_row_stats(sc.ctx, A, g)
        binding.sc_assign_lengths(sc.ctx, g, group, avg, Lmin, Lmax, L)
        binding.sc_matmul_prepared(sc.ctx, A, prepared[0], L, Lmax, params, P, C, ws)

    for _ in range(3):
        step_prepared()
    torch.cuda.synchronize()
    if graphed:
        graph_p = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph_p):
            step_prepared()
        step_prepared = graph_p.replay
        for _ in range(3):
            step_prepared()
        torch.cuda.synchronize()
    scdist.barrier()
    prepared_ms = scdist.max_over_ranks(sum(timed_steps(args.steps, step_prepared)), dev)
    status = sc.device_status()
    if status != 0:
        raise SystemExit("device status %d (%s) in the prepared-weights leg" % (status, binding.status_string(status)))
    binding.sc_weights_release(prepared[0])
    prepared = None
    clocks = sampler.stop() if rank == 0 else {}

    # ---- end to end: host buffers in, host result out, through the same calls ----------------------------
    e2e = None
    if not args.no_e2e:
        # Host buffers in, host result out, every step, through the same calls.  Three streams and two sets of
        # device buffers pipeline the steps the way a serving loop would: the copy-in of step i+1 and the
        # copy-out of step i-1 run on the copy engines while step i computes.  The timed region is one pair of
        # events around all K steps (every copy of every step lies inside it).
        A_pin = torch.from_numpy(A_h).pin_memory()
        W_pin = torch.from_numpy(W_h).pin_memory()
        C_pin = [torch.empty((w.M, w.N), dtype=torch.float32).pin_memory() for _ in range(2)]
        dA = [torch.empty_like(A) for _ in range(2)]
        dW = [torch.empty_like(W) for _ in range(2)]
        dC = [torch.empty_like(C) for _ in range(2)]
        s_in, s_out = torch.cuda.Stream(device=dev), torch.cuda.Stream(device=dev)

        def compute_on(b):
            def run():
                binding.sc_row_stats(sc.ctx, dA[b], g)
                binding.sc_assign_lengths(sc.ctx, g, group, avg, Lmin, Lmax, L)
                binding.sc_matmul(sc.ctx, dA[b], dW[b], L, Lmax, params, P, dC[b], ws)
            return run

        compute = [compute_on(0), compute_on(1)]
        if graphed:                                   # one captured graph per buffer set
            for b in range(2):
                gb = torch.cuda.CUDAGraph()
                with torch.cuda.graph(gb):
                    compute[b]()
                compute[b] = gb.replay
            stream = torch.cuda.current_stream()

        def e2e_run(n):
            ev_in = [torch.cuda.Event() for _ in range(n)]
            ev_done = [torch.cuda.Event() for _ in range(n)]
            ev_out = [torch.cuda.Event() for _ in range(n)]
            t0, t1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t0.record(stream)
            s_in.wait_event(t0)
            s_out.wait_event(t0)
            for i in range(n):
                b = i & 1
                with torch.cuda.stream(s_in):
                    if i >= 2:
                        s_in.wait_event(ev_done[i - 2])           # the buffers of step i-2 have been consumed
                    dA[b].copy_(A_pin, non_blocking=True)
                    dW[b].copy_(W_pin, non_blocking=True)
                    ev_in[i].record(s_in)
                stream.wait_event(ev_in[i])
                if i >= 2:
                    stream.wait_event(ev_out[i - 2])              # the result buffer of step i-2 has been read out
                compute[b]()
                ev_done[i].record(stream)
                with torch.cuda.stream(s_out):
                    s_out.wait_event(ev_done[i])
                    C_pin[b].copy_(dC[b], non_blocking=True)
                    ev_out[i].record(s_out)
            stream.wait_event(ev_out[n - 1])
            if n >= 2:
                stream.wait_event(ev_out[n - 2])
            t1.record(stream)
            torch.cuda.synchronize()
            return t0.elapsed_time(t1)

        e2e_run(3)
        scdist.barrier()
        e2e_ms = scdist.max_over_ranks(e2e_run(args.steps), dev)
        e2e = {"value": bitops_per_step * world_size * args.steps / (e2e_ms * 1e-3), "unit": UNIT,
               "h2d_bytes_per_step": int(A_h.nbytes + W_h.nbytes), "d2h_bytes_per_step": int(C_pin[0].numel() * 4),
               "ms_per_step": e2e_ms / args.steps,
               "how": "pinned host A and W copied in and C copied out every step; copies of neighbouring steps overlap "
                      "the compute on separate streams; the compute of a step is a replayed CUDA graph (one per buffer set) "
                      "unless --no-graph; one event pair around all steps (pipeline fill and drain included)"}

    if rank != 0:
        return

    value = bitops_per_step * world_size * args.steps / (total_ms * 1e-3)
    peaks = measured_peaks()
    sm_max = float(clocks.get("sm_max_mhz") or peaks.get("sm_max_mhz") or 1965.0)
    n_sm = torch.cuda.get_device_properties(dev).multi_processor_count
    core_avg_ms = statistics.mean(core_ms)
    achieved = bitops_per_step / (core_avg_ms * 1e-3)                    # stream bit-ops (= 1-bit MACs) per second
    alu_peak = POPC_PER_CLK_PER_SM * 32.0 * n_sm * sm_max * 1e6          # POPC-pipe bound of the ALU cores
    uses_tensor = args.core in (0, 4, 5) and w.K * Lmax <= (1 << 24)
    if uses_tensor:
        # Tensor contraction: one stream bit-op is one multiply-accumulate = 2 ops, run as 4-bit floating point
        # (e2m1, tcgen05.mma kind::mxf4).  Two denominators: (a) the measured bf16 burst figure x the nominal ratio of the
        # dense peaks (fp4 9 : bf16 2.25 PFLOP/s); (b) the issue rate of the core's own instruction, measured here by a
        # bare chain of MMAs (multiply-accumulates per clock per SM) x SMs x the maximum SM clock.  `peak` is the larger, so
        # that the headline fraction does not rest on a nominal ratio; both fractions are in the line.
        bf16 = peaks.get("bf16_tflops")
        peak_a = (bf16 if bf16 else 1590.0) * FP4_TO_BF16_NOMINAL
        mclk, macs = binding.sc_microbench(sc.ctx, 8, 4096)            # 128 x 192 x 64 block-scaled e2m1 MMAs
        mac_per_clk_sm = macs / (mclk * 1e6)
        peak_b = 2.0 * mac_per_clk_sm * n_sm * sm_max * 1e6 / 1e12
        peak_tops = max(peak_a, peak_b)
        ach = 2.0 * achieved / 1e12
        pair_ran = binding.sc_last_core_selected(sc.ctx) != 0          # the plan's choice between the two tensor-core kernels
        roofline = {
            "bound": "tensor",
            "kernel": ("core_umma_pair_kernel (tcgen05.mma.cta_group::2 kind::mxf4, 256 x 256 tiles on pairs of SMs, bits "
                       "expanded on chip)" if pair_ran else
                       "core_umma_kernel (tcgen05.mma kind::mxf4 on bits expanded on chip)"),
            "achieved": ach, "peak": peak_tops, "unit": "TFLOP/s", "frac": ach / peak_tops,
            "traffic": NCU_CORE_TRAFFIC_BYTES.get((w.name, "pair" if pair_ran else "umma")),
            "peak_source": ("the larger of (a) %s x %g (nominal fp4 : bf16) = %.0f TFLOP/s (`frac_vs_bf16_x4`) and (b) the measured "
                            "issue rate of the mxf4 MMA, %.0f MAC/clk/SM x %d SMs x %.0f MHz = %.0f TFLOP/s (`peak_issue_rate`, "
                            "`frac_vs_issue_rate`)"
                            % ("measured bf16 burst %.1f TFLOP/s (MEASURED_PEAKS.json)" % bf16 if bf16
                               else "fallback 1590 TFLOP/s bf16", FP4_TO_BF16_NOMINAL, peak_a, mac_per_clk_sm, n_sm, sm_max,
                               peak_b)),
            "frac_vs_bf16_x4": ach / peak_a, "peak_issue_rate": peak_b, "frac_vs_issue_rate": ach / peak_b,
            "mxf4_mac_per_clk_per_sm": mac_per_clk_sm,
            "core_ms": core_avg_ms, "bitops_per_s": achieved, "times_popc_alu_bound": achieved / alu_peak,
            "hbm_gbs_measured_peak": peaks.get("hbm_gbs"),
        }
        if clocks.get("sm_mhz"):
            roofline["frac_vs_issue_rate_at_sampled_clock"] = ach / (peak_b * clocks["sm_mhz"] / sm_max)
    else:
        roofline = {
            "bound": "alu", "kernel": "core_kernel (gate + popcount accumulation)",
            "achieved": achieved / 1e12, "peak": alu_peak / 1e12, "unit": "Tbitop/s", "frac": achieved / alu_peak,
            "traffic": NCU_CORE_TRAFFIC_BYTES.get((w.name, "alu")),
            "peak_source": "derived: 16 POPC/clk/SM x 32 bit-ops x %d SMs x %.0f MHz (max SM clock)" % (n_sm, sm_max),
            "core_ms": core_avg_ms, "hbm_gbs_measured_peak": peaks.get("hbm_gbs"),
        }
        if clocks.get("sm_mhz"):
            roofline["frac_at_sampled_clock"] = achieved / (alu_peak * clocks["sm_mhz"] / sm_max)
    if args.microbench:
        mb = {}
        for kind, name in ((0, "popc"), (4, "iadd3"), (2, "plain_mix_gates"), (3, "csa_mix_gates")):
            ms, words = binding.sc_microbench(sc.ctx, kind, 2000)
            mb[name + "_words_per_s"] = words / (ms * 1e-3)
        for kind, name in ((8, "tcgen05_mxf4_n192_mac_per_clk_per_sm"), (9, "tcgen05_mxf4_n256_mac_per_clk_per_sm")):
            mclk, macs = binding.sc_microbench(sc.ctx, kind, 4096)
            mb[name] = macs / (mclk * 1e6)
        roofline["microbench"] = mb

    cpu_baseline = None
    if not args.no_cpu_baseline:
        run, cb_bitops, sample, cores = oracle_sample(w, 128, 1024)
        dt = run()
        cpu_baseline = {"value": cb_bitops / dt, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample,
                        "seconds": dt}

    # ---- the other benchmark configurations, a few steps each (recorded numbers beside the headline) -------
    other = []
    if not args.no_configs and world_size == 1:
        del A, W, C, P, ws
        torch.cuda.empty_cache()
        for name in OTHER_CONFIGS:
            m = measure_workload(sc, dev, name, args.core, reps=3)
            core_rate = m["bitops"] / (m["core_ms"] * 1e-3)
            entry = {"workload": name, "mode": m["mode"], "mean_L": round(m["mean_L"], 2), "step_ms": m["step_ms"],
                     "core_ms": m["core_ms"], "prepared_step_ms": m["prepared_step_ms"],
                     "step_bitops_per_s": m["bitops"] / (m["step_ms"] * 1e-3), "core_bitops_per_s": core_rate}
            if m["tensor_core"] and roofline["bound"] == "tensor":
                entry["core_frac"] = 2.0 * core_rate / 1e12 / roofline["peak"]
                entry["core_frac_vs_issue_rate"] = 2.0 * core_rate / 1e12 / roofline["peak_issue_rate"]
                entry["core_frac_vs_bf16_x4"] = entry["core_frac"] / roofline["frac"] * roofline["frac_vs_bf16_x4"]
            else:
                entry["core_frac_alu"] = core_rate / alu_peak
            other.append(entry)
        status = sc.device_status()
        if status != 0:
            raise SystemExit("device status %d (%s) in the configs leg" % (status, binding.status_string(status)))

    mean_phase = {k: statistics.mean(p[k] for p in phases) for k in phases[0]}
    # achieved rates of the phases around the core (algorithmic bytes: fp32 operand read + packed planes written;
    # accumulators read + C written) and the SNG rate in generated stream bits per second
    ppq = 2 if w.mode == "unipolar" else 1
    enc_a_bytes = 4.0 * w.M * w.K + ppq * sum_L * w.K / 8.0
    enc_w_bytes = 4.0 * w.K * w.N + ppq * float(Lmax) * w.K * w.N / 8.0
    dec_bytes = 8.0 * w.M * w.N
    phase_rates = {
        "encode_a_gbs": enc_a_bytes / (mean_phase["encode_a"] * 1e-3) / 1e9,
        "encode_w_gbs": enc_w_bytes / (mean_phase["encode_w"] * 1e-3) / 1e9,
        "decode_gbs": dec_bytes / (mean_phase["decode"] * 1e-3) / 1e9,
        "encode_a_stream_bits_per_s": sum_L * w.K / (mean_phase["encode_a"] * 1e-3),
        "encode_w_stream_bits_per_s": float(Lmax) * w.K * w.N / (mean_phase["encode_w"] * 1e-3),
        "note": "encode is bound by the Philox arithmetic, not by HBM; encode_w includes the column popcount tables",
    }
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world_size, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None,
        "dtype": ("e2m1 tensor operands (1 stream bit -> 1 four-bit float) / exact fp32 integer accumulate" if uses_tensor
                  else "u32 packed stream bits / int32 popcounts"), "data": "synthetic",
        "config": {"workload": w.name, "M": w.M, "K": w.K, "N": w.N, "mode": w.mode,
                   "L": w.uniform_L if w.uniform_L else "policy avg %g in [%d,%d] group %d" % w.policy,
                   "mean_L": sum_L / w.M, "l2": "flushed between timed steps (256 MiB memset)",
                   "core_variant": args.core, "per_rank_batch": "%d x %d" % (w.M, w.K),
                   "launch": "CUDA graph of the step's kernels, replayed" if graphed else "kernel by kernel"},
        "equiv_mac_per_s": float(w.M) * w.N * w.K * world_size * args.steps / (total_ms * 1e-3),
        "e2e": e2e, "gpu_launches": int(launches), "clocks": clocks, "roofline": roofline,
        "cpu_baseline": cpu_baseline, "phase_ms": mean_phase, "phase_rates": phase_rates,
        "configs": other,
        "prepared_weights": {"value": bitops_per_step * world_size * args.steps / (prepared_ms * 1e-3), "unit": UNIT,
                             "ms_per_step": prepared_ms / args.steps,
                             "what": "same step through sc_matmul_prepared: the W-side encode is done once, outside "
                                     "the timed region (static weights); the headline value re-encodes W every step"},
    }
    print(json.dumps(line))


def oracle_free_sum_lengths(L, group, M):
    """Sum of the per-row lengths from the device-side group lengths (bookkeeping for the metric)."""
    import torch
    Lc = L.to(torch.int64).cpu()
    full = M // group
    total = int(Lc[:full].sum().item()) * group
    if M % group:
        total += int(Lc[full].item()) * (M % group)
    return total


if __name__ == "__main__":
    main()
