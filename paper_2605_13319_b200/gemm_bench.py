"""Stand-alone bandwidth test of the small-M weight-streaming GEMM (pipesd_gemm_run).

    python -m paper_2605_13319_b200.gemm_bench [--shapes 7b] [--m 9] [--iters 20] [--copies 0]

Each launch streams a different copy of the weight matrix so that no launch finds its weights in L2
(copies * N * K * 2 bytes is kept above 4x the 126 MB L2); durations are CUDA-event times on the launching stream.
Prints one line per shape: microseconds per launch and algorithmic GB/s (bf16 W once + fp32 x in + fp32 y out).
"""
from __future__ import annotations

import argparse
import json

import numpy as np

from . import binding, synth

SHAPE_SETS = {
    # (name, N, K)
    "7b": [("qkv", 12288, 4096), ("o", 4096, 4096), ("gate_up", 22016, 4096), ("down", 4096, 11008),
           ("lm_head", 32000, 4096)],
    "1b": [("qkv", 3072, 2048), ("o", 2048, 2048), ("gate_up", 16384, 2048), ("down", 2048, 8192),
           ("lm_head", 32000, 2048)],
    "8b": [("qkv", 6144, 4096), ("o", 4096, 4096), ("gate_up", 28672, 4096), ("down", 4096, 14336),
           ("lm_head", 128256, 4096)],
    "small": [("down", 4096, 11008)],
}


def main():
    import torch
    ap = argparse.ArgumentParser()
    ap.add_argument("--shapes", default="7b", choices=sorted(SHAPE_SETS))
    ap.add_argument("--m", type=int, default=9)
    ap.add_argument("--iters", type=int, default=20)
    ap.add_argument("--copies", type=int, default=0, help="weight copies to rotate through (0: enough to exceed L2 4x)")
    args = ap.parse_args()
    dev = torch.device("cuda", 0)
    M = args.m
    out = []
    for name, N, K in SHAPE_SETS[args.shapes]:
        wbytes = N * K * 2
        copies = args.copies or max(2, int(np.ceil(4 * 126e6 / wbytes)))
        W = torch.from_numpy(synth.normal_bf16((N, K), 0, 1, 0.02).view(np.int16)).to(dev)
        packed = [binding.gemm_pack(W) for _ in range(copies)]
        x = torch.from_numpy(synth.normal_f32((M, K), 0, 2)).to(dev)
        y = torch.empty((M, N), device=dev)
        scratch = binding.gemm_scratch(M, N, K, dev)
        for i in range(3):
            binding.gemm_run(packed[i % copies], x, y, scratch, N, K)
        torch.cuda.synchronize()
        evs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.iters)]
        st = torch.cuda.current_stream(dev)
        for i, (a, b) in enumerate(evs):
            a.record(st)
            binding.gemm_run(packed[i % copies], x, y, scratch, N, K)
            b.record(st)
        torch.cuda.synchronize()
        us = np.array([a.elapsed_time(b) for a, b in evs]) * 1e3
        alg = wbytes + 4 * M * K + 4 * M * N
        rec = {"gemm": name, "M": M, "N": N, "K": K, "us_median": float(np.median(us)), "us_min": float(us.min()),
               "GBps_median": alg / np.median(us) / 1e3, "copies": copies}
        print(json.dumps(rec), flush=True)
        out.append(rec)
        del packed, W
    return out


if __name__ == "__main__":
    main()
