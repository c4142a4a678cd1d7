#!/usr/bin/env python
"""Benchmark of the binarized-convolution hot path on B200.

One "step" is one pass of the whole path over one batch of synthetic input: for each of the four
ResNet-18 stage shapes (C = 64/128/256/512 at 56/28/14/7 pixels, 3x3, stride 1, pad 1 with value -1)
at batch 64: binarize + pack the fp32 activations, binary convolution with int32 output, and binary
convolution with the fused BN + sign + re-pack epilogue.  The headline value is the convolutions'
bit-operations (2 per bit pair) divided by the time of the whole step.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-extras]

Prints ONE JSON line (rank 0).  Under torchrun every rank runs the same per-GPU work on its own
seeded batch (weak scaling, no data-path collective); the time is the maximum over ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_1908_05858_b200 import synth  # noqa: E402

BATCH = 64
METRIC = "binary conv Gbit-ops/s"
UNIT = "Gbit-ops/s"
WORKLOAD = "binary 3x3 conv sweep, batch 64, (C,HW) in (64,56),(128,28),(256,14),(512,7): pack + bconv(int32) + bconv(bn,sign,pack)"


def conv_bitops(N, C, HW, O, k):
    return 2.0 * N * HW * HW * O * C * k * k


def step_bitops(batch):
    return sum(2 * conv_bitops(batch, C, HW, C, 3) for C, HW in synth.SWEEP_SHAPES)


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)), "source": "measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "source": "fallback"}


def measured_tensor_peak_tops():
    """Dense 4-bit (e2m1) tensor peak for the roofline: the measured bf16 burst peak x the nominal fp4 : bf16 ratio (4)."""
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"tops": float(d["bf16_tflops"]) * 4.0,
                "how": "measured bf16 burst peak %.0f TFLOP/s x 4 (nominal dense fp4 : bf16 ratio), of measured" % float(d["bf16_tflops"])}
    return {"tops": 1590.0 * 4.0, "how": "fallback bf16 peak 1590 TFLOP/s x 4 (nominal dense fp4 : bf16 ratio), of fallback"}


def bitop_peak_tbitops(sm_count, sm_mhz):
    """Carry-save bound of sum popcount(a xor w) on the B200 integer pipes: with one POPC (XU pipe, 16 lanes/clk/SM)
    and four logic ops (ALU pipe, 64 lanes/clk/SM) per two 32-bit word pairs both pipes are full at 32 word pairs
    per clock per SM; 32 bit pairs per word pair, 2 bit-ops per bit pair."""
    return sm_count * 32 * 32 * 2 * sm_mhz * 1e6 / 1e12


class ClockSampler:
    """Samples SM clock, power and throttle reasons through NVML from a background thread while the timed region runs."""

    def __init__(self, index, period_s=0.005):
        self.index, self.period = index, period_s
        self.samples, self.reasons, self.err = [], set(), None
        self._stop = None
        self._thread = None

    def start(self):
        import threading
        try:
            import pynvml
            pynvml.nvmlInit()
            uuid = None
            try:
                import torch
                uuid = str(torch.cuda.get_device_properties(self.index).uuid)
            except Exception:
                uuid = None
            h = None
            if uuid:
                try:
                    h = pynvml.nvmlDeviceGetHandleByUUID(("GPU-" + uuid) if not uuid.startswith("GPU-") else uuid)
                except Exception:
                    h = None
            if h is None:
                h = pynvml.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = float(pynvml.nvmlDeviceGetMaxClockInfo(h, pynvml.NVML_CLOCK_SM))
        except Exception as e:  # NVML not usable: report that instead of clocks
            self.err = "nvml unavailable: %s" % e
            return
        self._stop = threading.Event()
        R = pynvml
        masks = {"hw_slowdown": R.nvmlClocksThrottleReasonHwSlowdown,
                 "hw_thermal_slowdown": R.nvmlClocksThrottleReasonHwThermalSlowdown,
                 "sw_thermal_slowdown": R.nvmlClocksThrottleReasonSwThermalSlowdown,
                 "sw_power_cap": R.nvmlClocksThrottleReasonSwPowerCap}

        def loop():
            while not self._stop.is_set():
                try:
                    mhz = float(R.nvmlDeviceGetClockInfo(h, R.NVML_CLOCK_SM))
                    pw = R.nvmlDeviceGetPowerUsage(h) / 1000.0
                    bits = R.nvmlDeviceGetCurrentClocksThrottleReasons(h)
                    self.samples.append((mhz, pw))
                    for nm, m in masks.items():
                        if bits & m:
                            self.reasons.add(nm)
                except Exception as e:
                    self.err = str(e)
                    return
                self._stop.wait(self.period)

        self._thread = threading.Thread(target=loop, daemon=True)
        self._thread.start()

    def stop(self):
        if self._thread is not None:
            self._stop.set()
            self._thread.join(timeout=2)
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": [self.err or "no samples"]}
        sm = [m for m, _ in self.samples]
        return {"sm_mhz": statistics.median(sm), "sm_min_mhz": min(sm), "sm_max_mhz": self.max_mhz,
                "power_w_max": max(p for _, p in self.samples), "samples": len(sm), "reasons": sorted(self.reasons),
                "how": "NVML, every %.0f ms during the timed region" % (self.period * 1e3)}


# ---------------------------------------------------------------------------------------------------------------
def run_reference(args):
    """The oracle, as it stands, on the host cores: each step is a bounded sample (batch 2 per shape) of the
    workload, timed with the wall clock."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cores = oracle.max_threads()
    oracle.set_threads(cores)
    nb = 2
    cases = []
    for C, HW in synth.SWEEP_SHAPES:
        x, w = synth.conv_case(2, nb, C, HW, HW, C, 3, 3, salt=C)
        scale, shift = oracle.bn_fold(*synth.bn_params(synth.rng(2, 900 + C), C))
        cases.append((C, x, oracle.pack_weights(w), scale, shift))

    def step():
        for C, x, wp, scale, shift in cases:
            a = oracle.pack(x)
            oracle.bconv_bits(a, C, wp, (1, 1), (1, 1), -1)
            acc = oracle.bconv_bits(a, C, wp, (1, 1), (1, 1), -1)
            oracle.bn_sign_pack(acc, scale, shift)

    for _ in range(args.warmup):
        step()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        step()
    dt = time.perf_counter() - t0
    value = step_bitops(nb) * args.steps / dt / 1e9
    sample = "batch %d of each of the four shapes per step (the workload's batch is %d)" % (nb, BATCH)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u64 words / int32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "sample": sample},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ---------------------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the per-config extra measurements")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return

    import torch
    import torch.distributed as dist

    from paper_1908_05858_b200 import binding as B

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path (use --impl reference for the oracle)")
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    B.lib()
    dev = torch.device("cuda", local)
    sm_count = torch.cuda.get_device_properties(dev).multi_processor_count
    peaks = measured_peaks()
    warmup = max(args.warmup, 3)

    # ---- inputs: seeded, drawn on the host, resident in HBM before the timed region ------------------------------
    layers = []
    for C, HW in synth.SWEEP_SHAPES:
        x, w = synth.conv_case(2, BATCH, C, HW, HW, C, 3, 3, salt=C + 1000 * rank)
        g = synth.rng(2, 900 + C)
        bn = [torch.from_numpy(t).to(dev) for t in synth.bn_params(g, C)]
        scale, shift = B.bn_fold(*bn)
        xh = torch.from_numpy(x).pin_memory()
        L = {
            "C": C, "HW": HW, "x_host": xh, "x": xh.to(dev), "w": B.pack_weights(torch.from_numpy(w).to(dev)),
            "scale": scale, "shift": shift,
            "a": torch.empty((BATCH, HW, HW, (C + 63) // 64), dtype=torch.int64, device=dev),
            "out": torch.empty((BATCH, HW, HW, C), dtype=torch.int32, device=dev),
            "bits": torch.empty((BATCH, HW, HW, (C + 63) // 64), dtype=torch.int64, device=dev),
            "bitops": conv_bitops(BATCH, C, HW, C, 3),
        }
        L["wt"] = B.TcWeights(L["w"], C)  # the same weights expanded once for the tensor-core engine
        L["call_pack"] = B.prepare_pack(L["x"], L["a"])
        L["call_conv"] = {"popc": B.prepare_bconv2d(L["a"], C, L["w"], L["out"], (1, 1), (1, 1), -1, B.NHWC),
                          "tc": B.prepare_tc_bconv2d(L["a"], L["wt"], L["out"], (1, 1), (1, 1), -1, B.NHWC)}
        L["call_fused"] = {"popc": B.prepare_bconv2d_bn_sign_pack(L["a"], C, L["w"], L["scale"], L["shift"], L["bits"], (1, 1), (1, 1), -1),
                           "tc": B.prepare_tc_bconv2d_bn_sign_pack(L["a"], L["wt"], L["scale"], L["shift"], L["bits"], (1, 1), (1, 1), -1)}
        L["out_host"] = torch.empty(L["out"].shape, dtype=torch.int32).pin_memory()
        L["bits_host"] = torch.empty(L["bits"].shape, dtype=torch.int64).pin_memory()
        ws_bytes = B.binary_layer_host_workspace_bytes(BATCH, C, HW, HW, C, 3, 3, (1, 1), (1, 1), -1)
        L["ws"] = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        layers.append(L)
    # A second set of activation / output buffers with the same contents: consecutive steps alternate between the two
    # sets, so that whatever a step reads or writes was last touched two steps (about 390 MB of traffic) earlier and
    # has left the 126 MB L2; no flush kernel runs between steps.  Weights and BN vectors (1.3 MB) are shared.
    def twin(L):
        T = dict(L)
        C = L["C"]
        T["x"] = L["x"].clone()
        for key in ("a", "out", "bits"):
            T[key] = torch.empty_like(L[key])
        T["call_pack"] = B.prepare_pack(T["x"], T["a"])
        T["call_conv"] = {"popc": B.prepare_bconv2d(T["a"], C, L["w"], T["out"], (1, 1), (1, 1), -1, B.NHWC),
                          "tc": B.prepare_tc_bconv2d(T["a"], L["wt"], T["out"], (1, 1), (1, 1), -1, B.NHWC)}
        T["call_fused"] = {"popc": B.prepare_bconv2d_bn_sign_pack(T["a"], C, L["w"], L["scale"], L["shift"], T["bits"], (1, 1), (1, 1), -1),
                           "tc": B.prepare_tc_bconv2d_bn_sign_pack(T["a"], L["wt"], L["scale"], L["shift"], T["bits"], (1, 1), (1, 1), -1)}
        return T
    layer_sets = [layers, [twin(L) for L in layers]]

    def step(engine, convs_only=False, which=0):
        for L in layer_sets[which]:
            if not convs_only:
                L["call_pack"]()
            L["call_conv"][engine]()
            L["call_fused"][engine]()
    launches_per_step = 3 * len(layers)

    # The four shapes are independent layers: in the timed step each is its own branch (stream) of the step's CUDA graph,
    # pack -> convolution -> fused convolution in order inside a branch, so one shape's start-up and tail overlap the
    # others' work.  The same 12 kernels; the serial form is timed beside it.
    branch_streams = [torch.cuda.Stream() for _ in layers]

    def step_branched(engine, which=0):
        cur = torch.cuda.current_stream()
        for L, bs in zip(layer_sets[which], branch_streams):
            bs.wait_stream(cur)
            with torch.cuda.stream(bs):
                L["call_pack"]()
                L["call_conv"][engine]()
                L["call_fused"][engine]()
        for bs in branch_streams:
            cur.wait_stream(bs)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def capture(fn):
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                fn()
        torch.cuda.current_stream().wait_stream(side)
        return graph

    def timed_replays(graphs, n):
        """n replays back to back, alternating between the two buffer sets; returns the device time per replay in ms."""
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        graphs[1].replay()  # (the set that the first timed replay does not use)
        e0.record()
        for k in range(n):
            graphs[k % 2].replay()
        e1.record()
        torch.cuda.synchronize()
        return e0.elapsed_time(e1) / n

    for _ in range(warmup):
        for which in (0, 1):
            step("tc", which=which)
            step("popc", which=which)
    barrier()
    # each step is one CUDA-graph replay (one host call), so the timed loop is never host-bound
    g_step = {e: [capture(lambda e=e, w=w: step(e, which=w)) for w in (0, 1)] for e in ("tc", "popc")}
    # side by side, launches capped at half the chip each fill it better than launches that each take all of it
    B.tc_set_max_ctas(sm_count // 2)
    g_branched = [capture(lambda w=w: step_branched("tc", which=w)) for w in (0, 1)]
    B.tc_set_max_ctas(0)
    g_conv = {e: [capture(lambda e=e, w=w: step(e, convs_only=True, which=w)) for w in (0, 1)] for e in ("tc", "popc")}
    for _ in range(warmup):
        g_branched[0].replay()
        g_branched[1].replay()
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.05)
    barrier()
    host_t0 = time.perf_counter()
    # ---- the timed region: K steps with the faster (tensor-core) engine ------------------------------------------
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_start.record()
    for k in range(args.steps):
        g_branched[k % 2].replay()
    t_end.record()
    host_issue_ms = (time.perf_counter() - host_t0) * 1e3  # time the host needed to enqueue everything
    barrier()
    total_ms = torch.tensor([t_start.elapsed_time(t_end)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(total_ms, op=dist.ReduceOp.MAX)
    total_ms = float(total_ms.item())
    value = world * step_bitops(BATCH) * args.steps / (total_ms * 1e-3) / 1e9

    # ---- the dominant kernels on their own: the eight convolution launches of a step, per engine ------------------
    n_side = max(args.steps, 10)
    tc_ms, popc_ms = timed_replays(g_conv["tc"], n_side), timed_replays(g_conv["popc"], n_side)
    serial_step_ms = timed_replays(g_step["tc"], n_side)
    popc_step_ms = timed_replays(g_step["popc"], n_side)
    clocks = sampler.stop()
    conv_ops = step_bitops(BATCH)
    tensor_peak = measured_tensor_peak_tops()
    alu_peak = bitop_peak_tbitops(sm_count, peaks["sm_max_mhz"])
    roofline = {
        "bound": "tensor", "kernel": "bconv_tc_kernel (the 8 convolution launches of a step, one CUDA-graph replay)",
        "achieved": conv_ops / (tc_ms * 1e-3) / 1e12, "peak": tensor_peak["tops"], "unit": "TFLOP/s",
        "frac": conv_ops / (tc_ms * 1e-3) / 1e12 / tensor_peak["tops"], "peak_is": tensor_peak["how"],
        "traffic": 5.34e6, "traffic_is": "dram bytes of one N=64 C=256 28x28 launch (ncu, profiles/bconv_tc_kernel_N64_C256_HW28.md); most of its int32 output (51 MB, evict-first) is still in L2 when the kernel ends",
        "avg_launch_ms": tc_ms / 8, "conv_share_of_step": tc_ms / serial_step_ms,
        "conv_share_is": "the eight convolutions one after another / the 12 kernels one after another (%.4f ms)" % serial_step_ms,
        "note": "1 bit-op = 1 op: a +-1 multiply-add counts 2, as in FLOPs",
    }
    roofline_bitop = {
        "bound": "alu", "kernel": "bconv_kernel (integer pipes: xor + carry-save + popc), same 8 launches",
        "achieved": conv_ops / (popc_ms * 1e-3) / 1e12, "peak": alu_peak, "unit": "Tbit-ops/s",
        "frac": conv_ops / (popc_ms * 1e-3) / 1e12 / alu_peak,
        "peak_is": "ALU+XU carry-save bound at %d SMs x %.0f MHz (derived: 64 LOP3 lanes and 16 POPC lanes per clock and SM, carry-save halves the POPCs); the one-POPC-per-word-pair bound is half of it"
                   % (sm_count, peaks["sm_max_mhz"]),
        "traffic": 2.69e6, "traffic_is": "dram bytes of one N=64 C=256 28x28 launch (ncu, profiles/bconv_kernel_N64_C256_HW28.md)",
        "avg_launch_ms": popc_ms / 8,
        "step_value_with_this_engine": step_bitops(BATCH) / (popc_step_ms * 1e-3) / 1e9,
    }

    # ---- end to end through the host-buffer entry point ----------------------------------------------------------
    def e2e_step():
        for L in layers:
            B.binary_layer_host(L["x_host"], L["w"], L["ws"], (1, 1), (1, 1), -1, L["scale"], L["shift"],
                                out_host=L["out_host"], bits_host=L["bits_host"])
    e2e_steps = max(3, min(args.steps, 10))
    e2e_step()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(e2e_steps):
        e2e_step()
    e1.record()
    barrier()
    e2e_ms = torch.tensor([e0.elapsed_time(e1)], dtype=torch.float64, device=dev)
    if world > 1:
        dist.all_reduce(e2e_ms, op=dist.ReduceOp.MAX)
    e2e = {
        "value": world * step_bitops(BATCH) * e2e_steps / (float(e2e_ms.item()) * 1e-3) / 1e9, "unit": UNIT,
        "h2d_bytes_per_step": int(sum(L["x_host"].numel() * 4 for L in layers)),
        "d2h_bytes_per_step": int(sum(L["out_host"].numel() * 4 + L["bits_host"].numel() * 8 for L in layers)),
        "steps": e2e_steps, "api": "dabnn_binary_layer_host (pinned host buffers in and out)",
    }

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": total_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64 words / int32", "data": "synthetic",
        "config": {"workload": WORKLOAD, "batch_per_gpu": BATCH, "l2": "no flush: steps alternate between two buffer sets (about 390 MB touched between two uses of a buffer; L2 is 126 MB)",
                   "launch": "each step is one CUDA-graph replay of its 12 kernels: four branches, one per shape (pack -> conv int32 -> conv fused), that the GPU overlaps, tensor-engine launches capped at half the SMs each (dabnn_tc_set_max_ctas)",
                   "serial_ms_per_step": serial_step_ms,
                   "engine": "tensor-core engine (e2m1 tcgen05) for the timed steps; the integer-pipe engine is timed beside it (roofline_bitop)",
                   "parallelism": "replicas" if world > 1 else "single GPU"},
        "roofline": roofline, "roofline_bitop": roofline_bitop, "e2e": e2e,
        "gpu_launches": launches_per_step * args.steps, "clocks": clocks,
        "host_issue_ms_per_step": host_issue_ms / args.steps,
    }

    if rank == 0 and world == 1:
        if not args.no_cpu_baseline:
            result["cpu_baseline"] = cpu_baseline()
        if not args.no_extras:
            result["extras"] = extras(B, torch, dev, peaks, sm_count)
    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def cpu_baseline():
    """The oracle on the host cores, on a bounded sample of the same workload: whole steps at batch 32
    (half the workload's batch), repeated until about 10 s of wall time have passed."""
    import oracle
    cores = oracle.max_threads()
    oracle.set_threads(cores)
    nb = 32
    cases = []
    for C, HW in synth.SWEEP_SHAPES:
        x, w = synth.conv_case(2, nb, C, HW, HW, C, 3, 3, salt=C)
        scale, shift = oracle.bn_fold(*synth.bn_params(synth.rng(2, 900 + C), C))
        cases.append((C, x, oracle.pack_weights(w), scale, shift))
    t, reps = 0.0, 0
    while t < 10.0 and reps < 50:
        t0 = time.perf_counter()
        for C, x, wp, scale, shift in cases:
            a = oracle.pack(x)
            oracle.bconv_bits(a, C, wp, (1, 1), (1, 1), -1)
            acc = oracle.bconv_bits(a, C, wp, (1, 1), (1, 1), -1)
            oracle.bn_sign_pack(acc, scale, shift)
        t += time.perf_counter() - t0
        reps += 1
    return {"value": step_bitops(nb) * reps / t / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d steps at batch %d instead of %d (%.1f s of wall time on %d threads)" % (reps, nb, BATCH, t, cores)}


def extras(B, torch, dev, peaks, sm_count):
    """Per-configuration measurements beside the headline (each a few launches; CUDA events)."""
    out = {}

    def time_fn(fn, iters, flush=None):
        fn(); fn(); fn()
        torch.cuda.synchronize()
        ms = []
        for _ in range(iters):
            if flush is not None:
                flush.zero_()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); fn(); e1.record()
            torch.cuda.synchronize()
            ms.append(e0.elapsed_time(e1))
        return statistics.median(ms), min(ms)

    # bit-pack alone: fp32 NCHW 128x256x56x56 with ~1 % exact zeros (input 411 MB: cold by construction)
    x = torch.from_numpy(synth.pack_case()).to(dev)
    packed = torch.empty((128, 56, 56, 4), dtype=torch.int64, device=dev)
    med, best = time_fn(lambda: B.pack(x, B.NCHW, out=packed), 10)
    nbytes = x.numel() * 4 + packed.numel() * 8
    out["pack_128x256x56x56"] = {"ms": med, "GB/s": nbytes / med / 1e6, "frac_of_hbm_peak": nbytes / med / 1e6 / peaks["hbm_gbs"],
                                 "peak_GB/s": peaks["hbm_gbs"], "peak_source": peaks["source"], "bytes": nbytes,
                                 "how": "one launch per CUDA-event pair (includes the launch gap of a lone kernel)"}
    # the same launch ten times in one CUDA graph: the 411 MB input is larger than L2, so every launch reads DRAM, and
    # the gaps between a lone kernel and its events drop out
    s_pack = torch.cuda.Stream()
    with torch.cuda.stream(s_pack):
        B.pack(x, B.NCHW, out=packed)
        s_pack.synchronize()
        g_pack = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g_pack, stream=s_pack):
            for _ in range(10):
                B.pack(x, B.NCHW, out=packed)
        med10, _ = time_fn(g_pack.replay, 5)
    out["pack_128x256x56x56_back_to_back"] = {"ms": med10 / 10, "GB/s": nbytes / (med10 / 10) / 1e6,
                                              "frac_of_hbm_peak": nbytes / (med10 / 10) / 1e6 / peaks["hbm_gbs"]}
    del g_pack
    del x, packed

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    peak = bitop_peak_tbitops(sm_count, peaks["sm_max_mhz"])
    tpeak = measured_tensor_peak_tops()["tops"]
    for name, (N, C, HW, O, k, pad) in {"conv_256x256x28x28_3x3": (256, 256, 28, 256, 3, 1),
                                        "conv_256x512x14x14_1x1_to_2048": (256, 512, 14, 2048, 1, 0)}.items():
        g = torch.Generator(device=dev); g.manual_seed(5)
        a = torch.randint(-2**62, 2**62, (N, HW, HW, (C + 63) // 64), dtype=torch.int64, device=dev, generator=g)
        w = torch.randint(-2**62, 2**62, (O, k, k, (C + 63) // 64), dtype=torch.int64, device=dev, generator=g)
        o = torch.empty((N, HW, HW, O), dtype=torch.int32, device=dev)
        wt = B.TcWeights(w, C)
        ops = conv_bitops(N, C, HW, O, k)
        med, best = time_fn(lambda: B.bconv2d(a, C, w, (1, 1), (pad, pad), -1, B.NHWC, out=o), 10, flush)
        out[name] = {"int_pipes": {"ms": med, "Tbit-ops/s": ops / med / 1e9, "frac_of_bitop_peak": ops / med / 1e9 / peak}}
        med, best = time_fn(lambda: B.tc_bconv2d(a, wt, (1, 1), (pad, pad), -1, B.NHWC, out=o), 10, flush)
        out[name]["tensor"] = {"ms": med, "Tbit-ops/s": ops / med / 1e9, "frac_of_fp4_peak": ops / med / 1e9 / tpeak}
        # the same launch with the fused BN + sign + pack epilogue (what a stack of binary layers runs), back to back
        sc = torch.rand(O, device=dev) + 0.5
        sh = torch.randn(O, device=dev)
        bits = torch.empty((N, HW, HW, (O + 63) // 64), dtype=torch.int64, device=dev)
        fused_call = B.prepare_tc_bconv2d_bn_sign_pack(a, wt, sc, sh, bits, (1, 1), (pad, pad), -1)
        s_f = torch.cuda.Stream()
        with torch.cuda.stream(s_f):
            fused_call()
            s_f.synchronize()
            g_f = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g_f, stream=s_f):
                for _ in range(10):
                    fused_call()
            med10, _ = time_fn(g_f.replay, 5)
        out[name]["tensor_fused_back_to_back"] = {"ms": med10 / 10, "Tbit-ops/s": ops / (med10 / 10) / 1e9,
                                                  "frac_of_fp4_peak": ops / (med10 / 10) / 1e9 / tpeak}
        del a, w, o, wt, g_f, fused_call, bits

    # BGEMM against direct convolution, the comparison of the paper's Fig. 4, on config 5a: the im2col matrix of the packed
    # activations (padding taps hold the pad word) is materialised with torch slicing (plumbing, 58 MB of packed rows) and
    # multiplied by dabnn_bgemm; dabnn_bconv2d gathers the same rows on the fly (implicit BGEMM)
    N, C, HW, O = 256, 256, 28, 256
    g = torch.Generator(device=dev); g.manual_seed(9)
    a = torch.randint(-2**62, 2**62, (N, HW, HW, C // 64), dtype=torch.int64, device=dev, generator=g)
    w = torch.randint(-2**62, 2**62, (O, 3, 3, C // 64), dtype=torch.int64, device=dev, generator=g)

    def im2col():
        ap = torch.nn.functional.pad(a, (0, 0, 1, 1, 1, 1), value=-1)  # pad word: all bits set = -1 everywhere
        return torch.stack([ap[:, i:i + HW, j:j + HW, :] for i in range(3) for j in range(3)], dim=3).reshape(N * HW * HW, 9 * (C // 64))
    A = im2col()
    Bm = w.reshape(O, 9 * (C // 64))
    direct = B.bconv2d(a, C, w, (1, 1), (1, 1), -1, B.NHWC)
    same = bool((B.bgemm(A, Bm, 9 * C).reshape(N, HW, HW, O) == direct).all())
    ops = conv_bitops(N, C, HW, O, 3)
    t_gemm, _ = time_fn(lambda: B.bgemm(A, Bm, 9 * C), 5, flush)
    t_both, _ = time_fn(lambda: B.bgemm(im2col(), Bm, 9 * C), 5, flush)
    t_direct, _ = time_fn(lambda: B.bconv2d(a, C, w, (1, 1), (1, 1), -1, B.NHWC, out=direct), 5, flush)
    out["bgemm_vs_direct_256x256x28x28"] = {"identical": same, "bgemm_ms": t_gemm, "im2col_plus_bgemm_ms": t_both,
                                            "direct_ms": t_direct, "direct_Tbit-ops/s": ops / t_direct / 1e9,
                                            "bgemm_Tbit-ops/s": ops / t_gemm / 1e9,
                                            "note": "integer-pipe engine for both; im2col is torch slicing, not a tuned kernel"}
    del a, w, A, Bm, direct

    # batch-1 latency of the four sweep shapes (CUDA-graph replay of 50 launches)
    for C, HW in synth.SWEEP_SHAPES:
        g = torch.Generator(device=dev); g.manual_seed(7)
        a = torch.randint(-2**62, 2**62, (1, HW, HW, C // 64), dtype=torch.int64, device=dev, generator=g)
        w = torch.randint(-2**62, 2**62, (C, 3, 3, C // 64), dtype=torch.int64, device=dev, generator=g)
        o = torch.empty((1, HW, HW, C), dtype=torch.int32, device=dev)
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            for _ in range(3):
                B.bconv2d(a, C, w, (1, 1), (1, 1), -1, B.NHWC, out=o)
            s.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=s):
                for _ in range(50):
                    B.bconv2d(a, C, w, (1, 1), (1, 1), -1, B.NHWC, out=o)
            med, best = time_fn(graph.replay, 5)
        out["conv_batch1_C%d_%dx%d" % (C, HW, HW)] = {"us_per_conv": med * 1e3 / 50, "Tbit-ops/s": conv_bitops(1, C, HW, C, 3) / (med / 50) / 1e9}

    # Bi-Real Net 18: batch 128 (eager launches) and batch 1 (CUDA-graph replay)
    net = B.Bireal18(synth.bireal18_params())
    img = torch.from_numpy(synth.bireal18_images(128)).to(dev)
    logits = torch.empty((128, 1000), dtype=torch.float32, device=dev)
    med, best = time_fn(lambda: net.forward(img, logits), 5)
    out["bireal18_batch128"] = {"ms": med, "images/s": 128 / med * 1e3, "engine": "tensor-core engine on all 16 binary blocks"}
    s128 = torch.cuda.Stream()
    with torch.cuda.stream(s128):
        net.forward(img, logits)
        s128.synchronize()
        g128 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g128, stream=s128):
            for _ in range(4):
                net.forward(img, logits)
        med4, _ = time_fn(g128.replay, 5)
    out["bireal18_batch128_graph"] = {"ms": med4 / 4, "images/s": 128 / (med4 / 4) * 1e3,
                                      "launch": "four forward passes back to back in one CUDA graph"}
    del g128
    net_p = B.Bireal18(synth.bireal18_params(), engine="popc")
    med, best = time_fn(lambda: net_p.forward(img, logits), 5)
    out["bireal18_batch128_int_pipes"] = {"ms": med, "images/s": 128 / med * 1e3}
    del net_p
    img1, logits1 = img[:1].contiguous(), torch.empty((1, 1000), dtype=torch.float32, device=dev)
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        for _ in range(3):
            net.forward(img1, logits1)
        s.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=s):
            net.forward(img1, logits1)
        med, best = time_fn(graph.replay, 20)
    out["bireal18_batch1"] = {"ms": med, "images/s": 1e3 / med,
                              "launch": "CUDA graph replay of the 22 kernels (chained launches), one replay per event pair: latency of a lone forward"}
    with torch.cuda.stream(s):
        graph16 = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph16, stream=s):
            for _ in range(16):
                net.forward(img1, logits1)
        med16, _ = time_fn(graph16.replay, 10)
    out["bireal18_batch1_back_to_back"] = {"ms": med16 / 16, "images/s": 16e3 / med16,
                                           "launch": "sixteen batch-1 forwards back to back in one CUDA graph"}
    del graph16
    return out


if __name__ == "__main__":
    main()
