"""Runs a few launches of one dense-linear case, for use under a profiler.

Example (one Llama-7B-shaped QKV linear, 8 tokens, fast mode, 4 weight copies so that the
planes exceed the L2 capacity):

    python -m paper_2609_34380_b200.profile_case --layer qkv --M 8 --mode fast --copies 4 --iters 3

Grouped (MoE) case: --experts E routes --M tokens to two experts each (seeded) over E experts whose
matrices have --rows output rows (default: the layer's own) and the layer's K:

    python -m paper_2609_34380_b200.profile_case --family mixtral --layer gate_up --experts 8 --rows 7168 \
        --M 256 --mode fast --iters 3
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
    ap.add_argument("--fp8act", action="store_true", help="fast mode with FP8 activations (quantisation + FP8 linear)")
    ap.add_argument("--experts", type=int, default=0, help="> 0: grouped (MoE) linear over this many experts")
    ap.add_argument("--rows", type=int, default=0, help="grouped case: output rows per expert (0 = the layer's)")
    args = ap.parse_args()
    if args.experts > 0:
        return grouped_case(args)

    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n, k = SHAPES[args.family][args.layer]
    n = args.rows or n          # --rows overrides the layer's output rows (dense case too)
    enc_req = {"auto": dps.DPS_ENC_AUTO, "e4m3": dps.DPS_ENC_E4M3, "e5m2": dps.DPS_ENC_E5M2}[args.enc]
    mode = dps.DPS_MODE_FULL if args.mode == "full" else dps.DPS_MODE_FAST
    planes = []
    for c in range(args.copies):
        w = workloads.weights(n, k, 2001 + c, device=dev)
        planes.append(dps.dps_split_weights(w, enc_req))
        del w
    x = workloads.activations(args.M, k, 2011, device=dev)
    y = torch.empty((args.M, n), dtype=torch.float16, device=dev)
    if args.fp8act:
        q, scale = dps.dps_quantize_activations(x)

    def enqueue():
        for p, r, enc in planes:
            if args.fp8act:
                dps.dps_quantize_activations(x, q, scale)
                dps.dps_linear_fp8act(enc, q, scale, p, y)
            else:
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
    label = "fast+fp8act" if args.fp8act else args.mode
    print(f"{args.family}/{args.layer} N={n} K={k} M={args.M} {label}: {us:.2f} us/launch, "
          f"{nbytes / us / 1e3:.0f} GB/s, {2 * args.M * n * k / us / 1e6:.1f} TFLOP/s, status={dps.dps_stream_status()}")


def grouped_case(args) -> None:
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    n, k = SHAPES[args.family][args.layer]
    n = args.rows or n
    E, T = args.experts, args.M
    mode = dps.DPS_MODE_FULL if args.mode == "full" else dps.DPS_MODE_FAST
    ps, rs, encs = [], [], []
    for e in range(E):
        w = workloads.weights(n, k, 4001 + e, device=dev)
        p, r, enc = dps.dps_split_weights(w, dps.DPS_ENC_AUTO)
        ps.append(p), rs.append(r), encs.append(enc)
        del w
    P, R = torch.stack(ps), torch.stack(rs)
    del ps, rs
    x = workloads.activations(T, k, 4100, device=dev)
    tor, eor = workloads.top2_routing(T, E, 4200)
    tor_d, eor_d = torch.from_numpy(tor).to(dev), torch.from_numpy(eor).to(dev)
    y = torch.empty((2 * T, n), dtype=torch.float16, device=dev)
    ws = torch.empty(dps.dps_moe_workspace_bytes(2 * T, E, k), dtype=torch.uint8, device=dev)
    start, stop = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    for it in range(args.iters):
        if it == args.iters - 1:
            start.record()
        dps.dps_moe_linear(mode, encs, x, tor_d, eor_d, P, R if mode else None, y, ws)
    stop.record()
    torch.cuda.synchronize()
    us = 1e3 * start.elapsed_time(stop)
    nbytes = E * n * k * (2 if mode else 1) + 2 * T * k + 2 * 2 * T * n
    print(f"{args.family}/{args.layer} grouped E={E} N={n} K={k} tokens={T} {args.mode}: {us:.1f} us/call, "
          f"{nbytes / us / 1e3:.0f} GB/s, status={dps.dps_stream_status()}")


if __name__ == "__main__":
    main()
