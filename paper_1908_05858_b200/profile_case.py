"""Runs ONE kernel case a few times, for profiler captures and quick timing.

    python -m paper_1908_05858_b200.profile_case --case conv --N 64 --C 256 --HW 28 --O 256 --k 3 --iters 3

Cases: pack (fp32 NCHW -> packed), conv (int32 output), fused (BN + sign + pack epilogue),
bireal (Bi-Real Net 18 forward at batch N).  Inputs are seeded; the median CUDA-event time is printed.
"""
from __future__ import annotations

import argparse
import statistics

import torch

from . import binding as B
from . import synth


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--case", required=True, choices=["pack", "conv", "fused", "bireal"])
    ap.add_argument("--N", type=int, default=64)
    ap.add_argument("--C", type=int, default=256)
    ap.add_argument("--HW", type=int, default=28)
    ap.add_argument("--O", type=int, default=0)
    ap.add_argument("--k", type=int, default=3)
    ap.add_argument("--iters", type=int, default=3)
    ap.add_argument("--reps", type=int, default=1, help="launches per timed event pair")
    ap.add_argument("--graph", action="store_true", help="time a CUDA-graph replay of the `reps` launches")
    ap.add_argument("--variant", type=int, default=0)
    ap.add_argument("--tile", type=int, default=0)
    ap.add_argument("--engine", default="popc", choices=["popc", "tc"])
    a = ap.parse_args()
    O = a.O or a.C
    dev = torch.device("cuda", 0)
    B.set_conv_variant(a.variant)
    B.set_conv_tile(a.tile)
    pad = a.k // 2
    if a.case == "bireal":
        net = B.Bireal18(synth.bireal18_params())
        img = torch.from_numpy(synth.bireal18_images(a.N)).to(dev)
        fn = lambda: net.forward(img)
        work = None
    else:
        x, w = synth.conv_case(9, a.N, a.C, a.HW, a.HW, O, a.k, a.k)
        xd = torch.from_numpy(x).to(dev)
        wp = B.pack_weights(torch.from_numpy(w).to(dev))
        ap_ = B.pack(xd)
        scale = torch.ones(O, device=dev)
        shift = torch.zeros(O, device=dev)
        if a.case == "pack":
            out = torch.empty_like(ap_)
            fn = lambda: B.pack(xd, B.NCHW, out=out)
            work = ("GB/s", (xd.numel() * 4 + out.numel() * 8) / 1e9)
        elif a.case == "conv" and a.engine == "tc":
            out = torch.empty((a.N, a.HW, a.HW, O), dtype=torch.int32, device=dev)
            wt = B.TcWeights(wp, a.C)
            fn = lambda: B.tc_bconv2d(ap_, wt, (1, 1), (pad, pad), -1, B.NHWC, out=out)
            work = ("Tbit-ops/s", 2.0 * a.N * a.HW * a.HW * O * a.C * a.k * a.k / 1e12)
        elif a.case == "fused" and a.engine == "tc":
            out = torch.empty((a.N, a.HW, a.HW, (O + 63) // 64), dtype=torch.int64, device=dev)
            wt = B.TcWeights(wp, a.C)
            fn = lambda: B.tc_bconv2d_bn_sign_pack(ap_, wt, scale, shift, (1, 1), (pad, pad), -1, out=out)
            work = ("Tbit-ops/s", 2.0 * a.N * a.HW * a.HW * O * a.C * a.k * a.k / 1e12)
        elif a.case == "conv":
            out = torch.empty((a.N, a.HW, a.HW, O), dtype=torch.int32, device=dev)
            fn = lambda: B.bconv2d(ap_, a.C, wp, (1, 1), (pad, pad), -1, B.NHWC, out=out)
            work = ("Tbit-ops/s", 2.0 * a.N * a.HW * a.HW * O * a.C * a.k * a.k / 1e12)
        else:
            out = torch.empty((a.N, a.HW, a.HW, (O + 63) // 64), dtype=torch.int64, device=dev)
            fn = lambda: B.bconv2d_bn_sign_pack(ap_, a.C, wp, scale, shift, (1, 1), (pad, pad), -1, out=out)
            work = ("Tbit-ops/s", 2.0 * a.N * a.HW * a.HW * O * a.C * a.k * a.k / 1e12)
    fn()
    torch.cuda.synchronize()
    if a.graph:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            fn()
            side.synchronize()
            graph = torch.cuda.CUDAGraph()
            with torch.cuda.graph(graph, stream=side):
                for _ in range(a.reps):
                    fn()
        torch.cuda.current_stream().wait_stream(side)
        one, reps = fn, a.reps
        fn = graph.replay
        a.reps = 1
    ms = []
    for _ in range(a.iters):
        # `reps` launches back to back inside one event pair, so that launch latency is hidden behind the
        # previous launch's execution (a short kernel timed alone would measure the host, not the GPU)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(a.reps):
            fn()
        e1.record()
        torch.cuda.synchronize()
        ms.append(e0.elapsed_time(e1) / (reps if a.graph else a.reps))
    med = statistics.median(ms)
    line = "%s N=%d C=%d HW=%d O=%d k=%d: median %.4f ms" % (a.case, a.N, a.C, a.HW, O, a.k, med)
    if work:
        line += "  %.1f %s" % (work[1] / (med * 1e-3), work[0])
    print(line)


if __name__ == "__main__":
    main()
