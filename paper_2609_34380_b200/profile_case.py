"""Runs a few launches of one dense-linear case, for use under a profiler.

Example (one Llama-7B-shaped QKV linear, 8 tokens, fast mode, 4 weight copies so that the
planes exceed the L2 capacity):

    python -m paper_2609_34380_b200.profile_case --layer qkv --M 8 --mode fast --copies 4 --iters 3
"""
from __future__ import annotations

import argparse

import torch

import paper_2609_34380_b200 as dps
from paper_2609_34380_b200 import workloads

SHAPES = {"llama7b": workloads.LLAMA7B, "decoder70": workloads.DECODER70, "mixtral": workloads.MIXTRAL_EXPERT,
          "tiny": workloads.TINY}


def main() -> None:
    ap = argparse.ArgumentParser()
    ap.add_argument("--family", default="llama7b", choices=sorted(SHAPES))
    ap.add_argument("--layer", default="qkv")
    ap.add_argument("--M", type=int, default=8)
    ap.add_argument("--mode", default="fast", choices=["fast", "full"])
    ap.add_argument("--enc", default="auto", choices=["auto", "e4m3", "e5m2"])
    ap.add_argument("--copies", type=int, default=4)
    ap.add_argument("--iters", type=int, default=3)
    args = ap.parse_args()

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n, k = SHAPES[args.family][args.layer]
    enc_req = {"auto": dps.DPS_ENC_AUTO, "e4m3": dps.DPS_ENC_E4M3, "e5m2": dps.DPS_ENC_E5M2}[args.enc]
    mode = dps.DPS_MODE_FULL if args.mode == "full" else dps.DPS_MODE_FAST
    planes = []
    for c in range(args.copies):
        w = workloads.weights(n, k, 2001 + c, device=dev)
        planes.append(dps.dps_split_weights(w, enc_req))
        del w
    x = workloads.activations(args.M, k, 2011, device=dev)
    y = torch.empty((args.M, n), dtype=torch.float16, device=dev)
    def enqueue():
        for p, r, enc in planes:
            dps.dps_linear(mode, enc, x, p, r if mode else None, y)

    stream = torch.cuda.Stream()
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    with torch.cuda.stream(stream):
        enqueue()                                  # eager launches (these are what a profiler captures)
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            enqueue()
        for it in range(args.iters):
            if it == args.iters - 1:
                start.record(stream)
            graph.replay()
        stop.record(stream)
    torch.cuda.synchronize()
    us = 1e3 * start.elapsed_time(stop) / args.copies
    nbytes = n * k * (2 if mode else 1) + 2 * args.M * (n + k)
    print(f"{args.family}/{args.layer} N={n} K={k} M={args.M} {args.mode}: {us:.2f} us/launch, "
          f"{nbytes / us / 1e3:.0f} GB/s, {2 * args.M * n * k / us / 1e6:.1f} TFLOP/s, status={dps.dps_stream_status()}")


if __name__ == "__main__":
    main()
