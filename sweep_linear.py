"""Isolated fused base+LoRA linear sweep (the single-linear workload): times pm_linear_forward
(shrink + fused GEMM) per cell and reports algorithmic TFLOP/s.

  python sweep_linear.py                      # the whole grid
  python sweep_linear.py --k 768 --n 2304 --frames 256 --rank 16 --sets unif --iters 3

Cells: M = 197*B tokens, B in {16, 64, 256}; K->N in {768->2304, 768->3072, 3072->768}; 128 registered
adapters of rank in {8, 16, 32, 64}; 1-8 active adapters per frame, uniform or Zipf(1.2)-clustered;
plus a no-LoRA row per shape.  FLOPs counted: 2*M*K*N + 2*(K+N)*sum over rows of the active ranks.
"""
from __future__ import annotations

import argparse
import json
import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)


def run_cell(k_in, n_out, frames, rank, sets, iters, warmup=2, max_set=8, n_adapters=128):
    import torch
    import workloads as wl
    from paper_2507_14959_b200 import binding
    lora = sets != "none"
    cell = wl.linear_cell(k_in, n_out, frames, rank, clustered=(sets == "zipf"), n_adapters=n_adapters,
                          max_set=max_set)
    off = cell.set_offsets if lora else np.zeros(frames + 1, np.int32)
    ids = cell.set_ids if lora else np.zeros(0, np.int32)
    lin = binding.Linear(cell.w, cell.b, max_adapters=n_adapters, max_rank=rank, max_set=max_set,
                         max_frames=frames, tokens=cell.tokens, epilogue=0, dtype=0)
    if lora:
        for a in range(n_adapters):
            lin.register(a, rank, cell.scale, cell.A[a], cell.B[a])
    x = torch.from_numpy(cell.x).cuda().to(torch.bfloat16)
    rows = frames * cell.tokens
    y = torch.empty((rows, n_out), device="cuda", dtype=torch.bfloat16)
    for _ in range(warmup):
        lin.forward(x, frames, off, ids, y)
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(iters):
        lin.forward(x, frames, off, ids, y)
    e1.record()
    torch.cuda.synchronize()
    assert lin.status() == 0
    ms = e0.elapsed_time(e1) / iters
    active_rank = rank * len(ids)
    flops = 2.0 * rows * k_in * n_out + 2.0 * (k_in + n_out) * cell.tokens * active_rank
    lin.close()
    return {"k": k_in, "n": n_out, "frames": frames, "rank": rank if lora else 0, "sets": sets,
            "mean_active": len(ids) / frames, "ms": ms, "tflops": flops / ms / 1e9}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--k", type=int)
    ap.add_argument("--n", type=int)
    ap.add_argument("--frames", type=int)
    ap.add_argument("--rank", type=int, default=16)
    ap.add_argument("--sets", default="unif", choices=["unif", "zipf", "none"])
    ap.add_argument("--max-set", type=int, default=8)
    ap.add_argument("--iters", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=2)
    args = ap.parse_args()
    if args.k:
        print(json.dumps(run_cell(args.k, args.n, args.frames, args.rank, args.sets, args.iters, args.warmup,
                                  args.max_set)))
        return
    for k, n in [(768, 2304), (768, 3072), (3072, 768)]:
        for frames in (16, 64, 256):
            print(json.dumps(run_cell(k, n, frames, 16, "none", args.iters)), flush=True)
            for rank in (8, 16, 32, 64):
                for sets in ("unif", "zipf"):
                    print(json.dumps(run_cell(k, n, frames, rank, sets, args.iters)), flush=True)


if __name__ == "__main__":
    main()
