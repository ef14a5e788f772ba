#!/usr/bin/env python
"""Benchmark of the Polymorph hot path on B200: frames/s of the ViT-base production shape
(256 frames, 32 rank-16 adapters, 1-3 active adapters per frame).

A step = one pass of the whole hot path over one batch: routing plan, patch embed, 12 blocks
(LayerNorm, fused base+multi-LoRA linears, attention), final LayerNorm, heads + sigmoid + merge
(pm_forward) and Algorithm 2 selection on the base scores (pm_select).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--frames F]

With N > 1 (launched under torch.distributed.run) every rank runs the same batch shape on its own
GPU: frames are independent, so the path shards without any collective (weak scaling).
--impl reference times the CPU oracle on the host cores instead (a bounded sample per step).
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "frames/sec (ViT-base, 1-3 LoRA adapters/frame)"
UNIT = "frames/s"
# DRAM bytes per fused-GEMM launch from the ncu capture summarised in profiles/ (None until taken)
GEMM_DRAM_TRAFFIC_BYTES = 318e6     # mean over qkv / proj / fc1 / fc2 launches


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"bf16_tflops_sustained": float(p["bf16_tflops_sustained"]), "bf16_tflops": float(p["bf16_tflops"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops_sustained": 1400.0, "bf16_tflops": 1590.0, "hbm_gbs": 6650.0, "source": "fallback"}


def gemm_flops_per_step(w):
    """Algorithmic FLOPs of the fused linears of one step: per token 2*K*N for the base plus
    2*r*(K+N) per active adapter (Sec. 3.1), summed over qkv/proj/fc1/fc2 of every layer, plus the
    patch projection.  Padding, union-set masking and rank padding are not counted."""
    s = w.spec
    T, d, m, L = s.tokens, s.d, s.mlp, s.layers
    shapes = [(d, 3 * d), (d, d), (d, m), (m, d)]
    active_rank = sum(w.adapters[a].rank for a in w.set_ids)          # sum over frames of sum_a r_a
    F = w.n_frames
    base = sum(2 * k * n for k, n in shapes) * T * F * L
    # blocks an adapter really touches (its A/B pairs that are not None), per projection
    lora = 0
    for a in w.set_ids:
        ad = w.adapters[a]
        for i, (k, n) in enumerate(shapes):
            lora += 2 * (k + n) * T * ad.rank * sum(1 for l in range(L) if ad.A[l * 4 + i] is not None)
    patch = 2 * s.patch_dim * d * (T - 1) * F
    return base + lora + patch


def gemm_flops_per_step_branched(w, trunk_layers):
    """The same count for the branched arrangement (Fig. 2b): the trunk blocks once per frame, the
    remaining blocks once per branch (the base branch plus one per active adapter, each adapter
    alone in its branch)."""
    s = w.spec
    T, d, m, L = s.tokens, s.d, s.mlp, s.layers
    shapes = [(d, 3 * d), (d, d), (d, m), (m, d)]
    F = w.n_frames
    per_block = sum(2 * k * n for k, n in shapes) * T
    branches = F + len(w.set_ids)
    base = per_block * (F * trunk_layers + branches * (L - trunk_layers))
    lora = 0
    for a in w.set_ids:
        ad = w.adapters[a]
        for i, (k, n) in enumerate(shapes):
            lora += 2 * (k + n) * T * ad.rank * sum(1 for l in range(trunk_layers, L) if ad.A[l * 4 + i] is not None)
    return base + lora + 2 * s.patch_dim * d * (T - 1) * F


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed region runs."""
    Q = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,clocks_event_reasons.hw_slowdown,"
         "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
         "clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.Q}",
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        rows = [l for t, l in self.lines if t0 <= t <= t1 + 0.1] or [l for _, l in self.lines]
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for l in rows:
            f = [x.strip() for x in l.split(",")]
            if len(f) < 8:
                continue
            try:
                sm.append(float(f[0])); mx.append(float(f[1])); power.append(float(f[2]))
            except ValueError:
                continue
            for n, v in zip(names, f[4:8]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "power_w": float(np.median(power)) if power else None, "samples": len(sm),
                "reasons": sorted(reasons)}


def oracle_frames_per_s(w, n_sample):
    from oracle import polymorph_oracle as po
    rows = list(range(min(n_sample, w.n_frames)))
    sets = [w.sets()[r] for r in rows]
    import workloads as wl
    off, ids = wl.sets_to_csr(sets)
    t0 = time.perf_counter()
    po.forward(w.backbone, w.adapters, w.frames[rows], off, ids, w.spec.heads, w.spec.patch, w.spec.ln_eps,
               w.spec.n_classes)
    dt = time.perf_counter() - t0
    return len(rows) / dt, dt


def host_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 1) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return int(max(n))
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, rank):
    """The oracle as it stands, on the host cores: each step is a bounded sample of the workload."""
    if rank != 0:
        return
    import workloads as wl
    sample = 2
    w = wl.vit_base_batch(n_frames=max(sample, 2))
    for _ in range(args.warmup):
        oracle_frames_per_s(w, 1)
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_frames_per_s(w, sample)
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    cores = host_threads()
    out = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
           "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * dt / args.steps,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64",
           "data": "synthetic",
           "config": {"workload": "vit_base_batch (ViT-base 224x224, 32 rank-16 adapters, 1-3 per frame)",
                      "sample": f"{sample} frames per step on the host cores"},
           "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle",
                            "sample": f"{sample} frames per step, {args.steps} steps"},
           "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
           "gpu_launches": 0}
    print(json.dumps(out))


def run_streams(args, rank, world, dist):
    """Closed-loop streaming shape: 16 streams x 30 correlated 384x384 frames per GPU; a step is one
    time step (one frame per stream): pm_forward with the sets chosen at the previous step, then
    pm_select on the base scores.  The e2e leg copies each step's frames in and its scores out."""
    import torch
    import workloads as wl
    from paper_2507_14959_b200 import binding, shard, streaming
    T = 30
    if args.workload == "latency":
        S = 1
        w = wl.deit_tiny_stream(n_steps=T, n_streams=S)
        what = ("deit_tiny_stream: DeiT-tiny 224x224, ONE stream in closed loop (a step = one frame), 11 rank-16 "
                "query/value adapters on the last 2 blocks, 5 classes each")
    else:
        S = 16
        w = wl.vit_base_384_streams(n_streams=S, n_steps=T)
        what = ("vit_base_384_streams: ViT-base 384x384 (577 tokens), 16 streams/GPU in closed loop, 64 rank-16 "
                "adapters over 800 classes")
    mode = args.loop
    m = binding.model_from_workload(w, dtype=0, max_frames=S, max_set=8)
    m.set_cover(w.tau)
    K = w.spec.n_classes
    frames_host = torch.from_numpy(w.extra["stream_frames"]).to(torch.bfloat16).transpose(0, 1).contiguous().pin_memory()
    frames_dev = frames_host.cuda()                              # [T, S, 3, img, img]
    r = streaming.StreamRunner(m, S, K, len(w.adapters), 0.5, False, device_plan=mode != "host")
    stage = torch.empty_like(frames_dev[0])
    scores_host = torch.zeros((S, K)).pin_memory()
    stream = torch.cuda.current_stream()
    if mode == "graph":
        # one eager step sets every kernel up; then the step is recorded once per list-buffer parity
        r.reset()
        stage.copy_(frames_dev[0])
        r.step(stage)
        r.capture(stage)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def loop(n, e2e):
        for i in range(n):
            t = i % T
            if t == 0:
                r.reset()
            if mode == "graph":
                stage.copy_(frames_host[t] if e2e else frames_dev[t], non_blocking=True)
                sc, _ = r.step(stage) if t == 0 else r.step_graph()
            elif e2e:
                stage.copy_(frames_host[t], non_blocking=True)
                sc, _ = r.step(stage)
            else:
                sc, _ = r.step(frames_dev[t])
            if e2e:
                scores_host.copy_(sc, non_blocking=True)

    loop(max(args.warmup, 3), False)
    assert m.status() == 0
    out_ms = []
    launches = 0
    for e2e in (False, True):
        if e2e:
            loop(2, True)
        barrier()
        count = lambda: m.launch_count() + (r.replayed_launches if mode == "graph" else 0)
        n0 = count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        loop(args.steps, e2e)
        e1.record(stream)
        barrier()
        out_ms.append(e0.elapsed_time(e1))
        if not e2e:
            launches = count() - n0
    assert m.status() == 0
    ms, ms_e2e = shard.max_over_ranks(out_ms, device="cuda")
    if rank == 0:
        print(json.dumps({
            "metric": METRIC, "value": world * S * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": what + ", sets chosen by Algorithm 2 on the device",
                       "loop": {"host": "routing plan on the host (a device-to-host copy and a stream synchronisation per step)",
                                "device": "routing plan built on the device, no host synchronisation",
                                "graph": "routing plan built on the device; steps after a stream's first are CUDA-graph replays"}[mode],
                       "l2": "one step's activations fit the 126 MB L2; no flush" if args.workload == "latency"
                             else "one step touches ~0.2 GB of activations; no flush"},
            "latency_us_per_step": 1e3 * ms / args.steps,
            "e2e": {"value": world * S * args.steps / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(stage.numel() * 2), "d2h_bytes_per_step": int(scores_host.numel() * 4)},
            "gpu_launches": int(launches)}))
    m.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="polymorph", choices=["polymorph", "reference"])
    ap.add_argument("--frames", type=int, default=256, help="frames per GPU per step")
    ap.add_argument("--cpu-sample", type=int, default=16, help="frames of the CPU-baseline sample (0 = skip)")
    ap.add_argument("--lora-last", type=int, default=None,
                    help="batch workload only: adapters touch the last N blocks only (the paper's cheap "
                         "placement); default: all blocks, the headline configuration")
    ap.add_argument("--branched", action="store_true",
                    help="batch workload with --lora-last N only: the paper's arrangement (Fig. 2b) -- the first "
                         "layers-N blocks run once per frame, then the base model and every active adapter "
                         "continue as separate branches (pm_forward_branched)")
    ap.add_argument("--workload", default="batch", choices=["batch", "streams", "latency"],
                    help="batch: ViT-base 224x224, 256 frames (the headline); streams: ViT-base 384x384, 16 streams "
                         "in closed loop (forward -> Algorithm 2 -> next forward), one step = one frame per stream; "
                         "latency: DeiT-tiny, one stream in closed loop (the paper's embedded operating point)")
    ap.add_argument("--loop", default="graph", choices=["host", "device", "graph"],
                    help="streams / latency: where the routing plan of a step is built and whether steps are "
                         "CUDA-graph replays")
    args = ap.parse_args()
    args.warmup = max(args.warmup, 3) if args.impl == "polymorph" else args.warmup

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if args.impl == "reference":
        run_reference(args, rank)
        return

    import torch
    import workloads as wl
    from paper_2507_14959_b200 import binding, shard

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device (there is no CPU fallback)")
    torch.cuda.set_device(local_rank)
    # everything runs on a stream of its own: the legacy default stream cannot be recorded into CUDA graphs,
    # which the library does with its launch sequence once it has seen the same call twice
    torch.cuda.set_stream(torch.cuda.Stream())
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    if args.workload in ("streams", "latency"):
        run_streams(args, rank, world, dist)
        return

    w = wl.vit_base_batch(n_frames=args.frames, lora_last=args.lora_last)
    if args.branched and args.lora_last is None:
        raise SystemExit("--branched needs --lora-last N (adapters may not touch the shared trunk)")
    trunk = w.spec.layers - args.lora_last if args.branched else 0
    m = binding.model_from_workload(w, dtype=0, max_frames=w.n_frames + (len(w.set_ids) if args.branched else 0))
    m.set_cover(w.tau)
    F, K = w.n_frames, w.spec.n_classes
    frames_host = torch.from_numpy(w.frames).to(torch.bfloat16).pin_memory()
    frames_dev = frames_host.cuda()
    scores = torch.zeros((F, K), device="cuda")
    base = torch.zeros((F, K), device="cuda")
    scores_host = torch.zeros((F, K)).pin_memory()
    base_host = torch.zeros((F, K)).pin_memory()
    nw = (K + 31) // 32
    labels = torch.zeros((F, nw), dtype=torch.int32, device="cuda")
    sel = [(torch.zeros(F + 1, dtype=torch.int32, device="cuda"),
            torch.zeros(F * len(w.adapters), dtype=torch.int32, device="cuda")) for _ in range(2)]
    stream = torch.cuda.current_stream()

    def step(i, frames=None):
        if args.branched:
            m.forward_branched(frames_dev if frames is None else frames, w.set_offsets, w.set_ids, trunk, scores, base)
        else:
            m.forward(frames_dev if frames is None else frames, w.set_offsets, w.set_ids, scores, base)
        prev, nxt = sel[i % 2], sel[(i + 1) % 2]
        m.select(base, 0.5, False, i > 0, labels, prev[0], prev[1], nxt[0], nxt[1])

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    for i in range(args.warmup):
        step(i)
    assert m.status() == 0, "device status word set during warm-up"

    # ---- timed region: inputs resident in HBM --------------------------------------------
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else 0)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    n0 = m.launch_count()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    e0.record(stream)
    for i in range(args.steps):
        step(args.warmup + i)
    e1.record(stream)
    barrier()
    ms = e0.elapsed_time(e1)
    launches = m.launch_count() - n0
    # The same K steps once more with an event pair around every launch site (per-kernel times for
    # the roofline).  Kept out of the headline region: ~280 event records per step cost about 3 %.
    m.profile_enable(True)
    barrier()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    p0.record(stream)
    for i in range(args.steps):
        step(args.warmup + args.steps + i)
    p1.record(stream)
    barrier()
    t_wall1 = time.time()
    ms_profiled = p0.elapsed_time(p1)
    prof = m.profile_read()
    m.profile_enable(False)
    clocks = sampler.stop(t_wall0, t_wall1) if rank == 0 else None
    assert m.status() == 0, "device status word set during the timed region"

    # ---- end to end: host frames in, host scores out, copies inside the timed region ------
    # Every step copies its frames from pinned host memory and its scores back.  The input copy runs on
    # a second stream into one of two device buffers, so step i+1's frames travel while step i computes.
    copy_stream = torch.cuda.Stream()
    in_bufs = [frames_dev, torch.empty_like(frames_dev)]
    ready = [torch.cuda.Event(), torch.cuda.Event()]
    free = [torch.cuda.Event(), torch.cuda.Event()]
    for ev in free:
        ev.record(stream)

    def e2e_step(i):
        b = i % 2
        with torch.cuda.stream(copy_stream):
            copy_stream.wait_event(free[b])          # the step that last read this buffer is done
            in_bufs[b].copy_(frames_host, non_blocking=True)
            ready[b].record(copy_stream)
        stream.wait_event(ready[b])
        step(i, in_bufs[b])
        free[b].record(stream)
        scores_host.copy_(scores, non_blocking=True)
        base_host.copy_(base, non_blocking=True)

    for i in range(2):
        e2e_step(i)
    barrier()
    f0, f1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    f0.record(stream)
    for i in range(args.steps):
        e2e_step(i)
    f1.record(stream)
    barrier()
    ms_e2e = f0.elapsed_time(f1)

    ms, ms_e2e = shard.max_over_ranks([ms, ms_e2e], device="cuda")

    if rank == 0:
        peaks = measured_peaks()
        gemm_ms, gemm_sites = prof["gemm"]
        flops = (gemm_flops_per_step_branched(w, trunk) if args.branched else gemm_flops_per_step(w)) * args.steps
        achieved = flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
        peak = peaks["bf16_tflops_sustained"]
        out = {
            "metric": METRIC, "value": world * F * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": "vit_base_batch: ViT-base 224x224 (197 tokens), %d frames/GPU/step, 32 rank-16 "
                                   "adapters over 800 classes, 1-3 active adapters per frame (60/30/10 %%), "
                                   "forward + Algorithm 2 select" % F,
                       "frames_per_gpu": F, "l2": "activations (~0.9 GB/step) exceed the 126 MB L2; no flush",
                       "lora_blocks": "all 12" if args.lora_last is None else "last %d" % args.lora_last,
                       "arrangement": ("branched: %d shared blocks, then %d branches for %d frames" %
                                       (trunk, F + len(w.set_ids), F)) if args.branched else "one stream per frame"},
            "e2e": {"value": world * F * args.steps / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(frames_host.numel() * 2),
                    "d2h_bytes_per_step": int(scores_host.numel() * 4 + base_host.numel() * 4)},
            "gpu_launches": int(launches),
            "clocks": clocks,
            "roofline": {"bound": "tensor", "kernel": "lora_gemm_kernel (fused base + multi-LoRA linear)",
                         "achieved": achieved, "peak": peak, "unit": "TFLOP/s",
                         "frac": achieved / peak if peak else None,
                         "peak_source": "bf16_tflops_sustained of %s" % peaks["source"],
                         "launches_timed": gemm_sites, "avg_launch_ms": gemm_ms / max(gemm_sites, 1),
                         "timed_in": "a second pass of the same K steps with CUDA events around each launch site",
                         "traffic": None if args.branched else GEMM_DRAM_TRAFFIC_BYTES},
            "kernel_ms_per_step": {k: v[0] / args.steps for k, v in prof.items()},
            "profiled_pass_ms_per_step": ms_profiled / args.steps,
        }
        if args.cpu_sample > 0 and world == 1:
            v, dt = oracle_frames_per_s(w, args.cpu_sample)
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                                   "sample": f"{min(args.cpu_sample, F)} of the {F} frames, once ({dt:.1f} s)"}
        else:
            out["cpu_baseline"] = None
        print(json.dumps(out))
    m.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
