#!/usr/bin/env python
"""Benchmark of the binarized-convolution hot path on B200.

Workload: the large-batch configuration -- a binary 3x3 convolution (batch 256, 256 -> 256 channels, 28x28, stride 1,
pad 1 with value -1) and a binary 1x1 convolution (batch 256, 512 -> 2048 channels, 14x14).  One "step" is one pass of
the whole path over one batch of synthetic input, for each of the two layers: binarize + pack the fp32 activations,
binary convolution with int32 output, and binary convolution with the fused BN + sign + re-pack epilogue (6 kernels).
The headline value is the convolutions' bit-operations (2 per bit pair) divided by the time of the whole step, with the
xor + popcount kernels (the paper's method, on the integer pipes); the same step on the tensor-core engine, the pack
kernels' bandwidth and the Bi-Real Net 18 forward are reported in the same line.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--no-extras]
    python bench.py --case conv|fused|bireal_block|pack|bireal [--engine popc|tc] [--N ..] [--C ..] [--HW ..] [--O ..] [--k ..]

Prints ONE JSON line (rank 0).  Under torchrun every rank runs the same per-GPU work on its own seeded batch (weak
scaling, no data-path collective); times are the maximum over ranks.  `--case` runs one kernel case a few times (for
profiler captures and quick timings) and prints one text line instead.
"""
from __future__ import annotations

import argparse
import json
import os
import re
import statistics
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from paper_1908_05858_b200 import synth  # noqa: E402

BATCH = 256
# (name, C, HW, O, k, pad): the two layers of the large-batch configuration
LAYERS = (("conv3x3_256", 256, 28, 256, 3, 1), ("conv1x1_512_2048", 512, 14, 2048, 1, 0))
METRIC = "binary conv Gbit-ops/s (% of bit-op roofline); Bi-Real-18 images/s at batch 1/128"
UNIT = "Gbit-ops/s"
WORKLOAD = ("large-batch binary convolutions, batch 256: 3x3 256->256 at 28x28 (stride 1, pad 1, pad value -1) and "
            "1x1 512->2048 at 14x14; per layer pack + bconv(int32) + bconv(bn,sign,pack)")
REGIONS = 50  # the K-step timed region is repeated this many times (median and minimum reported)


def config_dict(world):
    return {"workload": WORKLOAD, "batch_per_gpu": BATCH,
            "l2": "inputs larger than L2: a step reads and writes 0.93 GB (L2 is 126 MB), no flush kernel",
            "parallelism": "replicas" if world > 1 else "single GPU"}


def conv_bitops(N, C, HW, O, k):
    return 2.0 * N * HW * HW * O * C * k * k


def step_bitops(batch):
    return sum(2 * conv_bitops(batch, C, HW, O, k) for _, C, HW, O, k, _ in LAYERS)


def conv_bytes(N, C, HW, O, k, fused):
    """Algorithmic HBM bytes of one convolution launch: packed activations + packed weights + the output."""
    cw = (C + 63) // 64
    out = N * HW * HW * ((O + 63) // 64) * 8 if fused else 4 * N * HW * HW * O
    return 8 * N * HW * HW * cw + 8 * O * k * k * cw + out


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as f:
            d = json.load(f)
        return {"hbm_gbs": float(d["hbm_gbs"]), "sm_max_mhz": float(d.get("sm_max_mhz", 1965.0)),
                "bf16_tflops": float(d["bf16_tflops"]), "bf16_tflops_sustained": float(d.get("bf16_tflops_sustained", d["bf16_tflops"])),
                "source": "of measured"}
    return {"hbm_gbs": 6650.0, "sm_max_mhz": 1965.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "source": "of fallback"}


def carry_save_peak_tbitops(sm_count, sm_mhz):
    """Carry-save bound of sum popcount(a xor w) on the B200 integer pipes: one POPC (XU pipe, 16 lanes/clk/SM) and
    three logic ops (ALU pipe, 64 lanes/clk/SM) per two 32-bit word pairs fill the XU pipe at 32 word pairs per clock
    per SM (ALU at 3/4); 32 bit pairs per word pair, 2 bit-ops per bit pair."""
    return sm_count * 32 * 32 * 2 * sm_mhz * 1e6 / 1e12


def popc_peak_tbitops(sm_count, sm_mhz):
    """One POPC per 32-bit word pair: 16 POPC lanes per clock and SM."""
    return sm_count * 16 * 32 * 2 * sm_mhz * 1e6 / 1e12


def profile_figure(filename, key):
    """A figure that a committed ncu summary under profiles/ states on a line `key: number` (None if absent)."""
    path = os.path.join(ROOT, "profiles", filename)
    if not os.path.exists(path):
        return None
    m = re.search(r"^%s:\s*([0-9.eE+]+)" % re.escape(key), open(path).read(), flags=re.M)
    return float(m.group(1)) if m else None


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
                "how": "NVML, every %.0f ms during the %d timed regions" % (self.period * 1e3, REGIONS)}


# ---------------------------------------------------------------------------------------------------------------
def oracle_cases(nb):
    import oracle
    cases = []
    for _, C, HW, O, k, pad in LAYERS:
        x, w = synth.conv_case(5, nb, C, HW, HW, O, k, k, salt=C)
        scale, shift = oracle.bn_fold(*synth.bn_params(synth.rng(5, 900 + C), O))
        cases.append((C, pad, x, oracle.pack_weights(w), scale, shift))
    return cases


def oracle_step(cases):
    import oracle
    for C, pad, x, wp, scale, shift in cases:
        a = oracle.pack(x)
        oracle.bconv_bits(a, C, wp, (1, 1), (pad, pad), -1)
        acc = oracle.bconv_bits(a, C, wp, (1, 1), (pad, pad), -1)
        oracle.bn_sign_pack(acc, scale, shift)


def run_reference(args):
    """The oracle, as it stands, on the host cores: each step is a bounded sample (batch 8 of each layer instead of 256)
    of the workload, timed with the wall clock."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import oracle
    cores = oracle.max_threads()
    oracle.set_threads(cores)
    nb = 8
    cases = oracle_cases(nb)
    for _ in range(args.warmup):
        oracle_step(cases)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_step(cases)
    dt = time.perf_counter() - t0
    value = step_bitops(nb) * args.steps / dt / 1e9
    sample = "batch %d of each layer per step (the workload's batch is %d), whole steps, %d threads" % (nb, BATCH, cores)
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3, "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": "u64 words / int32", "data": "synthetic",
        "config": config_dict(int(os.environ.get("WORLD_SIZE", "1"))),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


def cpu_baseline():
    """The oracle on the host cores, on a bounded sample of the same workload: whole steps at batch 8 of each layer
    (instead of 256) on all cores for about 8 s, and the same steps on one thread for about 6 s."""
    import oracle
    cores = oracle.max_threads()
    nb = 8
    cases = oracle_cases(nb)

    def timed(threads, budget_s):
        oracle.set_threads(threads)
        oracle_step(cases)
        t, reps = 0.0, 0
        while t < budget_s and reps < 200:
            t0 = time.perf_counter()
            oracle_step(cases)
            t += time.perf_counter() - t0
            reps += 1
        return step_bitops(nb) * reps / t / 1e9, reps, t

    v_all, r_all, t_all = timed(cores, 8.0)
    v_one, r_one, t_one = timed(1, 6.0)
    oracle.set_threads(cores)
    return {"value": v_all, "unit": UNIT, "cores": cores, "kind": "oracle",
            "sample": "%d whole steps at batch %d of each layer instead of %d (%.1f s of wall time on %d threads)" % (r_all, nb, BATCH, t_all, cores),
            "single_thread": {"value": v_one, "unit": UNIT, "cores": 1,
                              "sample": "%d of the same steps on one thread (%.1f s)" % (r_one, t_one)}}


# ---------------------------------------------------------------------------------------------------------------
def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-extras", action="store_true", help="skip the measurements beside the timed steps (pack, Bi-Real-18, ...)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--regions", type=int, default=REGIONS, help="repeats of the K-step timed region")
    # one kernel case, for profiler captures and quick timings
    ap.add_argument("--case", default=None, choices=["pack", "conv", "fused", "bireal_block", "bireal"])
    ap.add_argument("--engine", default="popc", choices=["popc", "tc"])
    ap.add_argument("--N", type=int, default=64)
    ap.add_argument("--C", type=int, default=256)
    ap.add_argument("--HW", type=int, default=28)
    ap.add_argument("--O", type=int, default=0)
    ap.add_argument("--k", type=int, default=3)
    ap.add_argument("--stride", type=int, default=1)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--reps", type=int, default=1, help="--case: launches per timed event pair")
    ap.add_argument("--graph", action="store_true", help="--case: time a CUDA-graph replay of the `reps` launches")
    ap.add_argument("--stem-module", action="store_true", help="--case bireal: the STEM module variant of the network")
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--tile", type=int, default=0)
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
        return
    if args.case:
        run_case(args)
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
    regions = max(args.regions, 1)

    # ---- inputs: seeded, drawn on the host, resident in HBM before the timed region ------------------------------
    layers = []
    for name, C, HW, O, k, pad in LAYERS:
        x, w = synth.conv_case(5, BATCH, C, HW, HW, O, k, k, salt=C + 1000 * rank)
        bn = [torch.from_numpy(t).to(dev) for t in synth.bn_params(synth.rng(5, 900 + C), O)]
        scale, shift = B.bn_fold(*bn)
        xh = torch.from_numpy(x).pin_memory()
        cw, ow = (C + 63) // 64, (O + 63) // 64
        L = {"name": name, "C": C, "HW": HW, "O": O, "k": k, "pad": pad, "x_host": xh, "x": xh.to(dev),
             "w": B.pack_weights(torch.from_numpy(w).to(dev)), "scale": scale, "shift": shift,
             "a": torch.empty((BATCH, HW, HW, cw), dtype=torch.int64, device=dev),
             "out": torch.empty((BATCH, HW, HW, O), dtype=torch.int32, device=dev),
             "bits": torch.empty((BATCH, HW, HW, ow), dtype=torch.int64, device=dev),
             "bitops": conv_bitops(BATCH, C, HW, O, k)}
        L["wt"] = B.TcWeights(L["w"], C)  # the same weights expanded once for the tensor-core engine
        st, pd = (1, 1), (pad, pad)
        L["call_pack"] = B.prepare_pack(L["x"], L["a"])
        L["call_conv"] = {"popc": B.prepare_bconv2d(L["a"], C, L["w"], L["out"], st, pd, -1, B.NHWC),
                          "tc": B.prepare_tc_bconv2d(L["a"], L["wt"], L["out"], st, pd, -1, B.NHWC)}
        L["call_fused"] = {"popc": B.prepare_bconv2d_bn_sign_pack(L["a"], C, L["w"], L["scale"], L["shift"], L["bits"], st, pd, -1),
                           "tc": B.prepare_tc_bconv2d_bn_sign_pack(L["a"], L["wt"], L["scale"], L["shift"], L["bits"], st, pd, -1)}
        layers.append(L)
    kernels_per_step = 3 * len(layers)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    def run_regions(engine, n_regions, k_steps):
        """n_regions timed regions of k_steps steps each, launched eagerly on the current stream with a CUDA event between
        all kernels.  Returns (ms of each region [max over ranks], {kernel name: mean ms per launch})."""
        names = []
        for L in layers:
            names += ["pack_" + L["name"], "conv_int32_" + L["name"], "conv_fused_" + L["name"]]
        ev = [[torch.cuda.Event(enable_timing=True) for _ in range(k_steps * kernels_per_step + 1)] for _ in range(n_regions)]
        for r in range(n_regions):
            e = ev[r]
            e[0].record()
            i = 1
            for _ in range(k_steps):
                for L in layers:
                    L["call_pack"](); e[i].record(); i += 1
                    L["call_conv"][engine](); e[i].record(); i += 1
                    L["call_fused"][engine](); e[i].record(); i += 1
        torch.cuda.synchronize()
        region_ms = torch.tensor([ev[r][0].elapsed_time(ev[r][-1]) for r in range(n_regions)], dtype=torch.float64, device=dev)
        if world > 1:
            dist.all_reduce(region_ms, op=dist.ReduceOp.MAX)
        per = {n: [] for n in names}
        for r in range(n_regions):
            for i in range(k_steps * kernels_per_step):
                per[names[i % kernels_per_step]].append(ev[r][i].elapsed_time(ev[r][i + 1]))
        return region_ms.cpu().tolist(), {n: statistics.fmean(v) for n, v in per.items()}

    for engine in ("popc", "tc"):
        run_regions(engine, 1, warmup)
    barrier()
    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.05)
    barrier()
    # ---- the timed regions: `regions` times K steps with the xor + popcount kernels ---------------------------------
    host_t0 = time.perf_counter()
    region_ms, per_kernel = run_regions("popc", regions, args.steps)
    host_ms = (time.perf_counter() - host_t0) * 1e3
    barrier()
    clocks = sampler.stop()
    med_ms, min_ms = statistics.median(region_ms), min(region_ms)
    value = world * step_bitops(BATCH) * args.steps / (med_ms * 1e-3) / 1e9
    # the same step on the tensor-core engine, timed the same way
    tc_regions = max(5, regions // 5)
    tc_region_ms, tc_per_kernel = run_regions("tc", tc_regions, args.steps)
    tc_med = statistics.median(tc_region_ms)

    # ---- rooflines ----------------------------------------------------------------------------------------------
    mhz = peaks["sm_max_mhz"]
    cs_peak, popc_peak = carry_save_peak_tbitops(sm_count, mhz), popc_peak_tbitops(sm_count, mhz)
    conv_names = [n for n in per_kernel if n.startswith("conv_")]
    ops_of = {}
    bytes_of = {}
    for L in layers:
        for form in ("int32", "fused"):
            ops_of["conv_%s_%s" % (form, L["name"])] = L["bitops"]
            bytes_of["conv_%s_%s" % (form, L["name"])] = conv_bytes(BATCH, L["C"], L["HW"], L["O"], L["k"], form == "fused")
        bytes_of["pack_" + L["name"]] = L["x"].numel() * 4 + L["a"].numel() * 8
    conv_ops = sum(ops_of[n] for n in conv_names)
    conv_ms = sum(per_kernel[n] for n in conv_names)
    achieved = conv_ops / (conv_ms * 1e-3) / 1e12
    sampled_mhz = clocks.get("sm_mhz") or mhz
    traffic = profile_figure("bconv_kernel_N256_C256_HW28_int32.md", "dram_bytes_per_launch")
    roofline = {
        "bound": "alu",
        "kernel": "bconv_kernel (xor + carry-save + popc on the integer pipes): the 4 convolution launches of a step, each timed "
                  "with CUDA events on the launching stream inside the timed regions",
        "achieved": achieved, "peak": cs_peak, "unit": "Tbit-ops/s", "frac": achieved / cs_peak,
        "peak_is": "derived: 16 POPC lanes (XU pipe) and 64 LOP3 lanes (ALU pipe) per clock and SM; the kernel's carry-save step is one POPC "
                   "and three logic ops per two 32-bit word pairs, so the XU pipe is full at 32 word pairs/clk/SM x %d SMs x %.0f MHz x 64 "
                   "bit-ops (ALU at 3/4); pipe rates %s (register-only micro-benchmark, profiles/ubench_int_pipes.md)" % (sm_count, mhz, peaks["source"]),
        "frac_at_sampled_clock": achieved / carry_save_peak_tbitops(sm_count, sampled_mhz),
        "popc_roofline": {"peak": popc_peak, "frac": achieved / popc_peak,
                          "peak_is": "one POPC per 32-bit word pair: 16 POPC/clk/SM x %d SMs x 32 bits x 2 x %.0f MHz" % (sm_count, mhz)},
        "avg_launch_ms": conv_ms / len(conv_names),
        "traffic": traffic,
        "traffic_is": "dram__bytes_read.sum + dram__bytes_write.sum of one conv_int32_conv3x3_256 launch at the bench's full size "
                      "(profiles/bconv_kernel_N256_C256_HW28_int32.md); algorithmic bytes of that launch: %d" % bytes_of["conv_int32_conv3x3_256"],
        "per_launch": {n: {"ms": per_kernel[n], "Tbit-ops/s": ops_of[n] / per_kernel[n] / 1e9,
                           "frac": ops_of[n] / per_kernel[n] / 1e9 / cs_peak, "frac_of_popc_roofline": ops_of[n] / per_kernel[n] / 1e9 / popc_peak}
                       for n in conv_names},
        "hbm_kernels": {n: {"ms": per_kernel[n], "GB/s": bytes_of[n] / per_kernel[n] / 1e6,
                            "frac": bytes_of[n] / per_kernel[n] / 1e6 / peaks["hbm_gbs"], "peak": peaks["hbm_gbs"], "peak_is": peaks["source"]}
                        for n in per_kernel if n.startswith("pack_")},
        "note": "1 bit-op = 1 op: a +-1 multiply-add counts 2, as in FLOPs",
    }
    # the tensor-core engine (not the bit-op method: its own bounds, never a % of the bit-op roofline)
    fp4_peak = peaks["bf16_tflops_sustained"] * 4.0
    tc_launch = {}
    for n in conv_names:
        ms = tc_per_kernel[n]
        t_hbm = bytes_of[n] / (peaks["hbm_gbs"] * 1e9) * 1e3
        t_tensor = ops_of[n] / (fp4_peak * 1e12) * 1e3
        bound = "hbm" if t_hbm >= t_tensor else "tensor"
        tc_launch[n] = {"ms": ms, "Tops/s": ops_of[n] / ms / 1e9, "bound": bound, "bound_ms": max(t_hbm, t_tensor),
                        "frac": max(t_hbm, t_tensor) / ms,
                        "GB/s": bytes_of[n] / ms / 1e6}
    roofline["tensor_engine"] = {
        "value": world * step_bitops(BATCH) * args.steps / (tc_med * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": tc_med / args.steps,
        "regions": tc_regions, "kernel": "bconv_tc_kernel (bits expanded on chip to e2m1, tcgen05.mma kind::mxf4, TMEM accumulators)",
        "per_launch": tc_launch,
        "bounds_are": "per launch the slower of HBM (algorithmic bytes / %.0f GB/s %s) and the tensor pipe (ops / %.0f Tops/s = sustained bf16 "
                      "peak %.0f x 4, the nominal dense fp4 : bf16 ratio, %s)" % (peaks["hbm_gbs"], peaks["source"], fp4_peak,
                                                                                 peaks["bf16_tflops_sustained"], peaks["source"]),
        "pack_ms": {n: tc_per_kernel[n] for n in tc_per_kernel if n.startswith("pack_")},
    }

    # ---- end to end through the host-buffer entry point ----------------------------------------------------------
    for L in layers:
        L["out_host"] = torch.empty(L["out"].shape, dtype=torch.int32).pin_memory()
        L["bits_host"] = torch.empty(L["bits"].shape, dtype=torch.int64).pin_memory()
        ws_bytes = B.binary_layer_host_workspace_bytes(BATCH, L["C"], L["HW"], L["HW"], L["O"], L["k"], L["k"], (1, 1), (L["pad"], L["pad"]), -1)
        L["ws"] = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)

    def e2e_step():
        for L in layers:
            B.binary_layer_host(L["x_host"], L["w"], L["ws"], (1, 1), (L["pad"], L["pad"]), -1, L["scale"], L["shift"],
                                out_host=L["out_host"], bits_host=L["bits_host"])
    e2e_steps = max(3, min(args.steps, 5))
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
        "steps": e2e_steps, "ms_per_step": float(e2e_ms.item()) / e2e_steps,
        "api": "dabnn_binary_layer_host (pinned host buffers in and out, copies inside the timed region; xor + popcount kernels)",
    }
    for L in layers:
        for key in ("out_host", "bits_host", "ws", "x_host"):
            L.pop(key)

    result = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": warmup,
        "ms_per_step": med_ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "u64 words / int32", "data": "synthetic", "config": config_dict(world),
        "roofline": roofline, "e2e": e2e,
        "gpu_launches": kernels_per_step * args.steps * regions, "clocks": clocks,
        "timed": {"regions": regions, "steps_per_region": args.steps, "region_ms_median": med_ms, "region_ms_min": min_ms,
                  "total_ms": sum(region_ms), "host_ms": host_ms,
                  "how": "each region = K steps launched eagerly (6 kernels per step, a CUDA event between kernels); value and ms_per_step "
                         "come from the median region; engine = xor + popcount kernels on the integer pipes"},
    }
    if rank == 0 and world == 1:
        del layers
        torch.cuda.empty_cache()
        if not args.no_extras:
            bireal, extra = extras(B, torch, dev, peaks, sm_count)
            result["bireal18"] = bireal
            result["roofline"]["bireal18"] = bireal
            result["roofline"]["pack_128x256x56x56"] = extra.pop("pack_128x256x56x56_back_to_back")
            result["extras"] = extra
        if not args.no_cpu_baseline:
            result["cpu_baseline"] = cpu_baseline()
    if rank == 0:
        print(json.dumps(result))
    if world > 1:
        dist.destroy_process_group()


def time_fn(torch, fn, iters, flush=None):
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


def graph_of(torch, fn, reps):
    s = torch.cuda.Stream()
    s.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(s):
        fn()
        s.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g, stream=s):
            for _ in range(reps):
                fn()
    torch.cuda.current_stream().wait_stream(s)
    return g


def extras(B, torch, dev, peaks, sm_count):
    """Measurements beside the timed steps (each a few launches; CUDA events): the Bi-Real Net 18 forward at batch 1 and
    128, the bit-pack configuration, the batch-64 and batch-1 sweeps, BGEMM against direct convolution."""
    out = {}

    # Bi-Real Net 18: batch 128 (eager launches and four forwards per CUDA graph) and batch 1 (CUDA-graph replay)
    net = B.Bireal18(synth.bireal18_params())
    img = torch.from_numpy(synth.bireal18_images(128)).to(dev)
    logits = torch.empty((128, 1000), dtype=torch.float32, device=dev)
    med, best = time_fn(torch, lambda: net.forward(img, logits), 10)
    g128 = graph_of(torch, lambda: net.forward(img, logits), 4)
    med4, _ = time_fn(torch, g128.replay, 10)
    del g128
    net_p = B.Bireal18(synth.bireal18_params(), engine="popc")
    med_p, _ = time_fn(torch, lambda: net_p.forward(img, logits), 5)
    del net_p
    img1, logits1 = img[:1].contiguous(), torch.empty((1, 1000), dtype=torch.float32, device=dev)
    g1 = graph_of(torch, lambda: net.forward(img1, logits1), 1)
    med1, _ = time_fn(torch, g1.replay, 30)
    g16 = graph_of(torch, lambda: net.forward(img1, logits1), 16)
    med16, _ = time_fn(torch, g16.replay, 10)
    del g1, g16
    # the STEM module variant (Section 2.3, Table 2 second row; structure = this library's reading of the missing figure)
    pst = dict(synth.bireal18_params())
    pst["stem_module"] = synth.stem_module_params()
    net_s = B.Bireal18(pst)
    gs128 = graph_of(torch, lambda: B.bireal18_forward_stem_module(net_s, img, logits), 4)
    med_s4, _ = time_fn(torch, gs128.replay, 10)
    gs1 = graph_of(torch, lambda: B.bireal18_forward_stem_module(net_s, img1, logits1), 1)
    med_s1, _ = time_fn(torch, gs1.replay, 30)
    del gs128, gs1, net_s
    flag = B.last_device_flag()
    bireal = {
        "unit": "images/s",
        "batch_128": {"images_per_s": 128 / (med4 / 4) * 1e3, "ms": med4 / 4,
                      "launch": "four forward passes back to back in one CUDA graph; tensor-core engine on the 16 binary blocks",
                      "eager_ms": med, "eager_images_per_s": 128 / med * 1e3,
                      "xor_popcount_kernels_only_ms": med_p, "xor_popcount_kernels_only_images_per_s": 128 / med_p * 1e3},
        "batch_1": {"images_per_s": 1e3 / med1, "ms": med1,
                    "launch": "CUDA-graph replay of the 22 chained kernels, one replay per event pair: latency of a lone forward",
                    "back_to_back_ms": med16 / 16, "back_to_back_images_per_s": 16e3 / med16},
        "with_stem_module": {"batch_128": {"images_per_s": 128 / (med_s4 / 4) * 1e3, "ms": med_s4 / 4},
                             "batch_1": {"images_per_s": 1e3 / med_s1, "ms": med_s1},
                             "note": "Section 2.3: the 7x7 convolution and max-pool replaced by the STEM module (a reading of the missing figure); same launch forms as above"},
        "device_flag_after": flag,
    }
    del net, img, logits

    # bit-pack alone: fp32 NCHW 128x256x56x56 with ~1 % exact zeros (input 411 MB: cold by construction)
    x = torch.from_numpy(synth.pack_case()).to(dev)
    packed = torch.empty((128, 56, 56, 4), dtype=torch.int64, device=dev)
    med, best = time_fn(torch, lambda: B.pack(x, B.NCHW, out=packed), 10)
    nbytes = x.numel() * 4 + packed.numel() * 8
    out["pack_128x256x56x56"] = {"ms": med, "GB/s": nbytes / med / 1e6, "frac_of_hbm_peak": nbytes / med / 1e6 / peaks["hbm_gbs"],
                                 "how": "one launch per CUDA-event pair (includes the launch gap of a lone kernel)"}
    g_pack = graph_of(torch, lambda: B.pack(x, B.NCHW, out=packed), 10)
    med10, _ = time_fn(torch, g_pack.replay, 5)
    out["pack_128x256x56x56_back_to_back"] = {"bound": "hbm", "ms": med10 / 10, "GB/s": nbytes / (med10 / 10) / 1e6,
                                              "frac": nbytes / (med10 / 10) / 1e6 / peaks["hbm_gbs"], "peak": peaks["hbm_gbs"],
                                              "peak_is": peaks["source"], "bytes": nbytes,
                                              "how": "ten launches in one CUDA graph; the 411 MB input is larger than L2, so every launch reads DRAM"}
    del g_pack, x, packed

    # the batch-64 sweep of the four stage shapes (pack + conv int32 + conv fused each), per engine, as one CUDA graph
    cs_peak = carry_save_peak_tbitops(sm_count, peaks["sm_max_mhz"])
    sweep = []
    for C, HW in synth.SWEEP_SHAPES:
        g = torch.Generator(device=dev); g.manual_seed(5)
        xs = torch.randn((64, C, HW, HW), device=dev, generator=g)
        w = torch.randint(-2**62, 2**62, (C, 3, 3, C // 64), dtype=torch.int64, device=dev, generator=g)
        sweep.append({"C": C, "x": xs, "w": w, "wt": B.TcWeights(w, C), "a": torch.empty((64, HW, HW, C // 64), dtype=torch.int64, device=dev),
                      "o": torch.empty((64, HW, HW, C), dtype=torch.int32, device=dev), "sc": torch.rand(C, device=dev) + 0.5,
                      "sh": torch.randn(C, device=dev), "bits": torch.empty((64, HW, HW, C // 64), dtype=torch.int64, device=dev)})
    sweep_ops = sum(2 * conv_bitops(64, C, HW, C, 3) for C, HW in synth.SWEEP_SHAPES)

    def sweep_step(engine):
        for S in sweep:
            B.pack(S["x"], B.NCHW, out=S["a"])
            if engine == "tc":
                B.tc_bconv2d(S["a"], S["wt"], (1, 1), (1, 1), -1, B.NHWC, out=S["o"])
                B.tc_bconv2d_bn_sign_pack(S["a"], S["wt"], S["sc"], S["sh"], (1, 1), (1, 1), -1, out=S["bits"])
            else:
                B.bconv2d(S["a"], S["C"], S["w"], (1, 1), (1, 1), -1, B.NHWC, out=S["o"])
                B.bconv2d_bn_sign_pack(S["a"], S["C"], S["w"], S["sc"], S["sh"], (1, 1), (1, 1), -1, out=S["bits"])
    for engine in ("popc", "tc"):
        gs = graph_of(torch, lambda: sweep_step(engine), 4)
        m, _ = time_fn(torch, gs.replay, 10)
        out["sweep_batch64_%s" % engine] = {"ms_per_step": m / 4, "Tbit-ops/s": sweep_ops / (m / 4) / 1e9,
                                            "frac_of_carry_save_bound": sweep_ops / (m / 4) / 1e9 / cs_peak if engine == "popc" else None}
        del gs
    del sweep

    flush = torch.empty(256 << 20, dtype=torch.uint8, device=dev)
    # the paper's NC1HWC2 activation layout (C2 = 128 bits; Section 2.1.2, last paragraph) beside channel-packed NHWC words on
    # the 3x3 layer: pack and convolution each, same kernels, same integers
    xs, ws = synth.conv_case(5, 256, 256, 28, 28, 256, 3, 3, salt=256)
    xd = torch.from_numpy(xs).to(dev)
    wpk = B.pack_weights(torch.from_numpy(ws).to(dev))
    lay = {}
    outs = {}
    for name, pl in (("nhwc_words", B.PACKED_NHWC), ("nc1hwc2", B.PACKED_NC1HWC2)):
        ap = B.pack_as(xd, pl)
        o32 = torch.empty((256, 28, 28, 256), dtype=torch.int32, device=dev)
        t_pack, _ = time_fn(torch, lambda: B.pack_as(xd, pl, out=ap), 10)
        t_conv, _ = time_fn(torch, lambda: B.bconv2d_from(ap, pl, 256, wpk, (1, 1), (1, 1), -1, B.NHWC, out=o32), 10, flush)
        lay[name] = {"pack_ms": t_pack, "conv_ms": t_conv, "conv_Tbit-ops/s": conv_bitops(256, 256, 28, 256, 3) / t_conv / 1e9}
        outs[name] = o32
    lay["identical"] = bool((outs["nhwc_words"] == outs["nc1hwc2"]).all())
    out["layout_nc1hwc2_vs_nhwc_words_256x256x28x28"] = lay
    del xd, wpk, outs, ap, o32
    # BGEMM against direct convolution, the comparison of the paper's Fig. 4, on the 3x3 layer: the im2col matrix of the packed
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
    t_gemm, _ = time_fn(torch, lambda: B.bgemm(A, Bm, 9 * C), 5, flush)
    t_both, _ = time_fn(torch, lambda: B.bgemm(im2col(), Bm, 9 * C), 5, flush)
    t_direct, _ = time_fn(torch, lambda: B.bconv2d(a, C, w, (1, 1), (1, 1), -1, B.NHWC, out=direct), 5, flush)
    out["bgemm_vs_direct_256x256x28x28"] = {"identical": same, "bgemm_ms": t_gemm, "im2col_plus_bgemm_ms": t_both,
                                            "direct_ms": t_direct, "direct_Tbit-ops/s": ops / t_direct / 1e9,
                                            "bgemm_Tbit-ops/s": ops / t_gemm / 1e9,
                                            "note": "im2col is torch slicing, not a tuned kernel"}
    del a, w, A, Bm, direct

    # batch-1 latency of the four sweep shapes (CUDA-graph replay of 50 launches)
    for C, HW in synth.SWEEP_SHAPES:
        g = torch.Generator(device=dev); g.manual_seed(7)
        a = torch.randint(-2**62, 2**62, (1, HW, HW, C // 64), dtype=torch.int64, device=dev, generator=g)
        w = torch.randint(-2**62, 2**62, (C, 3, 3, C // 64), dtype=torch.int64, device=dev, generator=g)
        o = torch.empty((1, HW, HW, C), dtype=torch.int32, device=dev)
        graph = graph_of(torch, lambda: B.bconv2d(a, C, w, (1, 1), (1, 1), -1, B.NHWC, out=o), 50)
        med, best = time_fn(torch, graph.replay, 5)
        out["conv_batch1_C%d_%dx%d" % (C, HW, HW)] = {"us_per_conv": med * 1e3 / 50, "Tbit-ops/s": conv_bitops(1, C, HW, C, 3) / (med / 50) / 1e9}
        del graph
    return bireal, out


# ---------------------------------------------------------------------------------------------------------------
def run_case(a):
    """Runs ONE kernel case a few times and prints the median CUDA-event time: what the ncu commands under profiles/ run."""
    import torch

    from paper_1908_05858_b200 import binding as B

    O = a.O or a.C
    dev = torch.device("cuda", 0)
    B.set_conv_variant(a.variant)
    B.set_conv_tile(a.tile)
    pad = a.k // 2
    st = (a.stride, a.stride)
    OHW = (a.HW + 2 * pad - a.k) // a.stride + 1
    ops = 2.0 * a.N * OHW * OHW * O * a.C * a.k * a.k / 1e12
    work = ("Tbit-ops/s", ops)
    if a.case == "bireal":
        params = dict(synth.bireal18_params())
        if a.stem_module:
            params["stem_module"] = synth.stem_module_params()
        net = B.Bireal18(params, engine="popc" if a.engine == "popc" else "auto")
        img = torch.from_numpy(synth.bireal18_images(a.N)).to(dev)
        logits = torch.empty((a.N, 1000), dtype=torch.float32, device=dev)
        fn = (lambda: B.bireal18_forward_stem_module(net, img, logits)) if a.stem_module else (lambda: net.forward(img, logits))
        work = ("images/ms", a.N * 1e-3)
    else:
        x, w = synth.conv_case(9, a.N, a.C, a.HW, a.HW, O, a.k, a.k)
        xd = torch.from_numpy(x).to(dev)
        wp = B.pack_weights(torch.from_numpy(w).to(dev))
        ap_ = B.pack(xd)
        scale = torch.rand(O, device=dev) + 0.5
        shift = torch.randn(O, device=dev)
        wt = B.TcWeights(wp, a.C) if a.engine == "tc" else None
        if a.case == "pack":
            out = torch.empty_like(ap_)
            fn = lambda: B.pack(xd, B.NCHW, out=out)
            work = ("GB/s", (xd.numel() * 4 + out.numel() * 8) / 1e9)
        elif a.case == "conv":
            out = torch.empty((a.N, OHW, OHW, O), dtype=torch.int32, device=dev)
            fn = ((lambda: B.tc_bconv2d(ap_, wt, st, (pad, pad), -1, B.NHWC, out=out)) if wt else
                  (lambda: B.bconv2d(ap_, a.C, wp, st, (pad, pad), -1, B.NHWC, out=out)))
        elif a.case == "fused":
            out = torch.empty((a.N, OHW, OHW, (O + 63) // 64), dtype=torch.int64, device=dev)
            fn = ((lambda: B.tc_bconv2d_bn_sign_pack(ap_, wt, scale, shift, st, (pad, pad), -1, out=out)) if wt else
                  (lambda: B.bconv2d_bn_sign_pack(ap_, a.C, wp, scale, shift, st, (pad, pad), -1, out=out)))
        else:  # bireal_block: the residual epilogue, in place on the fp32 stream as the network runs it
            res = torch.randn((a.N, OHW, OHW, O), device=dev)
            call = B.prepare_bireal_block(ap_, a.C, wp, wt, scale, shift, res, st, (pad, pad), -1)
            fn = call
    fn()
    torch.cuda.synchronize()
    reps = a.reps
    if a.graph:
        g = graph_of(torch, fn, a.reps)
        fn, per = g.replay, a.reps
        reps = 1
    else:
        per = a.reps
    ms = []
    for _ in range(a.iters):
        # `reps` launches back to back inside one event pair, so that launch latency is hidden behind the
        # previous launch's execution (a short kernel timed alone would measure the host, not the GPU)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1) / per)
    med = statistics.median(ms)
    print("%s engine=%s N=%d C=%d HW=%d O=%d k=%d stride=%d: median %.4f ms  %.1f %s" %
          (a.case, a.engine, a.N, a.C, a.HW, O, a.k, a.stride, med, work[1] / (med * 1e-3), work[0]))


if __name__ == "__main__":
    main()
