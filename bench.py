#!/usr/bin/env python
"""Benchmark of the Polymorph hot path on B200: frames/s of the ViT-base production shape
(256 frames, 32 rank-16 adapters, 1-3 active adapters per frame).

A step = one pass of the whole hot path over one batch: routing plan, patch embed, 12 blocks
(LayerNorm, fused base+multi-LoRA linears, attention), final LayerNorm, heads + sigmoid + merge
(pm_forward) and Algorithm 2 selection on the base scores (pm_select).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--impl reference] [--frames F]
                  [--sets-change P] [--device-sets] [--workload batch|streams|latency]

Three timed passes: (1) the headline, exactly K steps with the inputs resident in HBM; (2) the
roofline pass, the same steps once more with a CUDA-event pair around every launch site, continued
until it has run for --roofline-seconds so that the per-kernel figures are sustained ones; (3) end to
end, K steps whose frames come from pinned host memory and whose scores go back to it.

With N > 1 (launched under torch.distributed.run) every rank runs the same batch shape on its own
GPU: frames are independent, so the path shards without any collective (weak scaling).
--impl reference times the CPU oracle on the host cores instead (a bounded sample per step).
"""
from __future__ import annotations

import argparse
import json
import math
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

UNIT = "frames/s"
METRICS = {
    "batch": "frames/sec (ViT-base, 1-3 LoRA adapters/frame)",
    "streams": "frames/sec (ViT-base 384x384, 16 streams in closed loop, adapter sets chosen by Algorithm 2)",
    "latency": "frames/sec (DeiT-tiny, one stream in closed loop, adapter sets chosen by Algorithm 2)",
}


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        with open(path) as fh:
            p = json.load(fh)
        return {"bf16_tflops_sustained": float(p["bf16_tflops_sustained"]), "bf16_tflops": float(p["bf16_tflops"]),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    return {"bf16_tflops_sustained": 1400.0, "bf16_tflops": 1590.0, "hbm_gbs": 6650.0, "source": "fallback"}


def dram_traffic(kernel):
    """DRAM bytes per launch of `kernel` from the ncu capture recorded in profiles/ (None if there is
    no line for it, i.e. the kernel has changed since its counters were taken)."""
    path = os.path.join(ROOT, "profiles", "dram_traffic_per_launch.txt")
    try:
        with open(path) as fh:
            for line in fh:
                f = line.split()
                if len(f) >= 3 and not line.startswith("#") and f[0] == kernel:
                    return {"bytes": float(f[1]), "source": f[2]}
    except OSError:
        pass
    return None


# --------------------------------------------------------------------------------------
# algorithmic work (Sec. 3.1): what the method itself computes, no padding, no recomputation
# --------------------------------------------------------------------------------------
def linear_shapes(s):
    return [(s.d, 3 * s.d), (s.d, s.d), (s.d, s.mlp), (s.mlp, s.d)]


def linear_flops(spec, adapters, frame_sets, first_layer=0, rows_per_layer=None):
    """FLOPs of the fused linears for frames with the given adapter sets, split into the base product
    x W, the LoRA expand t B (both run in the fused GEMM kernel) and the LoRA shrink x A (its own
    kernel): per token 2 K N, 2 r N and 2 r K per active adapter that really touches the linear.
    rows_per_layer[l] = frames (branches) block l runs on; default: every frame in every block."""
    T, L = spec.tokens, spec.layers
    shapes = linear_shapes(spec)
    F = len(frame_sets)
    rows = rows_per_layer or [F] * L
    base = sum(2 * k * n for k, n in shapes) * T * sum(rows)
    expand = shrink = 0
    for st in frame_sets:
        for a in st:
            ad = adapters[a]
            for i, (k, n) in enumerate(shapes):
                touched = sum(1 for l in range(first_layer, L) if ad.A[l * 4 + i] is not None)
                expand += 2 * ad.rank * n * T * touched
                shrink += 2 * ad.rank * k * T * touched
    patch = 2 * spec.patch_dim * spec.d * (T - 1) * F
    return {"base": base, "expand": expand, "shrink": shrink, "patch": patch}


def hbm_bytes(spec, n_frames, n_adapter_rows, n_adapters, n_shrink_linears_per_layer=4):
    """Algorithmic bytes per launch of the bandwidth-bound kernels (bf16 activations)."""
    T, d, m, K = spec.tokens, spec.d, spec.mlp, spec.n_classes
    M = n_frames * T
    return {
        # the shrink streams x once per adapted linear: d (qkv) + d (proj) + d (fc1) + mlp (fc2) columns
        "shrink_per_layer": M * (3 * d + m) * 2,
        "attention": M * (3 * d + d) * 2,                    # q, k, v in; output
        "row_stats": M * d * 2,                              # read only
        "layernorm": 2 * M * d * 2,                          # read + write
        # final LayerNorm of the CLS rows, base head and adapter heads: rows, weights, two score arrays
        "heads": n_frames * d * 2 + n_frames * d * 4 * 2 + d * K * 2 + n_adapter_rows * d * 2 + 2 * n_frames * K * 4,
        # scores, cover tables, label bit sets (read + write), the two id lists
        "select": n_frames * K * 4 + K * 4 + K * 8 * ((n_adapters + 63) // 64) + 2 * n_frames * ((K + 31) // 32) * 4
                  + 4 * (n_frames + 1) * 4,
    }


class ClockSampler:
    """Samples nvidia-smi clocks and throttle reasons while the timed regions run."""
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
            time.sleep(0.3)
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append((time.time(), line.strip()))

    def stop(self):
        if not self.proc:
            return
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()

    def window(self, t0, t1):
        if not self.proc:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
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


def oracle_frames_per_s(w, frames, sets):
    from oracle import polymorph_oracle as po
    import workloads as wl
    off, ids = wl.sets_to_csr(sets)
    t0 = time.perf_counter()
    po.forward(w.backbone, w.adapters, frames, off, ids, w.spec.heads, w.spec.patch, w.spec.ln_eps,
               w.spec.n_classes)
    dt = time.perf_counter() - t0
    return len(sets) / dt, dt


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
        oracle_frames_per_s(w, w.frames[:1], w.sets()[:1])
    t0 = time.perf_counter()
    for _ in range(args.steps):
        oracle_frames_per_s(w, w.frames[:sample], w.sets()[:sample])
    dt = time.perf_counter() - t0
    value = sample * args.steps / dt
    cores = host_threads()
    out = {"impl": "reference", "metric": METRICS["batch"], "value": value, "unit": UNIT, "n_gpus": args.gpus,
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


def roofline_block(prof, steps, flops, bytes_, peaks, clocks, traffic, n_layers, region_s):
    """Per-kernel figures of the roofline pass.  `prof` = {class: (ms, launch sites)} over `steps`
    steps; flops = linear_flops(...) per step; bytes_ = hbm_bytes(...) per launch."""
    def tf(fl, ms):
        return fl * steps / (ms * 1e-3) / 1e12 if ms > 0 else None

    def gbs(by, ms, sites):
        return by * sites / (ms * 1e-3) / 1e9 if ms > 0 and sites > 0 else None

    gemm_ms, gemm_sites = prof["gemm"]
    shr_ms, shr_sites = prof["shrink"]
    sustained, burst = peaks["bf16_tflops_sustained"], peaks["bf16_tflops"]
    gemm_tf = tf(flops["base"] + flops["expand"] + flops["patch"], gemm_ms)
    fused_tf = tf(flops["base"] + flops["expand"] + flops["patch"] + flops["shrink"], gemm_ms + shr_ms)
    scale = (clocks["sm_max_mhz"] / clocks["sm_mhz"]) if clocks and clocks.get("sm_mhz") else None
    roof = {
        "bound": "tensor", "kernel": "fused base + multi-LoRA linear (shrink kernel + lora_gemm kernel)",
        "achieved": fused_tf, "peak": sustained, "unit": "TFLOP/s",
        "frac": fused_tf / sustained if fused_tf else None,
        "peak_source": "bf16_tflops_sustained of %s (the pass runs for seconds)" % peaks["source"],
        "frac_of_burst_peak": fused_tf / burst if fused_tf else None, "burst_peak": burst,
        "achieved_at_max_clock": fused_tf * scale if fused_tf and scale else None,
        "flops_per_step": flops, "ms_per_step": {"gemm": gemm_ms / steps, "shrink": shr_ms / steps},
        "gemm_only": {"achieved": gemm_tf, "frac": gemm_tf / sustained if gemm_tf else None,
                      "frac_of_burst_peak": gemm_tf / burst if gemm_tf else None,
                      "flops": "base + expand + patch projection; shrink excluded",
                      "launches_timed": gemm_sites, "avg_launch_ms": gemm_ms / max(gemm_sites, 1)},
        "timed_in": "%d steps (%.2f s) with CUDA events around each launch site, after the headline pass"
                    % (steps, region_s),
        "traffic": traffic["bytes"] if traffic else None,
        "traffic_source": traffic["source"] if traffic else None,
    }
    hbm = peaks["hbm_gbs"]
    entries = {}
    for name, cls, per_launch in (("shrink", "shrink", None), ("attention", "attention", bytes_["attention"]),
                                  ("row_stats", "layernorm", bytes_["row_stats"]), ("heads", "heads", bytes_["heads"]),
                                  ("select", "select", bytes_["select"])):
        ms, sites = prof[cls]
        if sites == 0:
            entries[name] = None
            continue
        if name == "shrink":
            total = bytes_["shrink_per_layer"] * n_layers * steps       # x once per adapted linear
            ach = total / (ms * 1e-3) / 1e9
            per = total / sites
        else:
            ach = gbs(per_launch, ms, sites)
            per = per_launch
        entries[name] = {"bound": "hbm", "achieved": ach, "peak": hbm, "unit": "GB/s", "frac": ach / hbm,
                         "bytes_per_launch": per, "launches_timed": sites, "avg_launch_us": 1e3 * ms / sites}
    return roof, entries


def run_streams(args, rank, world, dist, local_rank):
    """Closed-loop shapes.  streams: ViT-base 384x384 (577 tokens), 16 streams x 30 correlated frames per
    GPU; latency: DeiT-tiny, one stream.  A step is one time step (one frame per stream): the forward
    with the sets chosen at the previous step, then pm_select on the base scores.  The e2e leg copies
    each step's frames in and its scores out."""
    import torch
    import workloads as wl
    from paper_2507_14959_b200 import binding, shard, streaming
    T = 30
    if args.workload == "latency":
        S = 1
        w = wl.deit_tiny_stream(n_steps=T, n_streams=S)
        what = ("deit_tiny_stream: DeiT-tiny 224x224 (197 tokens), ONE stream in closed loop (a step = one frame), "
                "11 rank-16 query/value adapters on the last 2 blocks, 5 classes each")
    else:
        S = 16
        w = wl.vit_base_384_streams(n_streams=S, n_steps=T)
        what = ("vit_base_384_streams: ViT-base 384x384 (577 tokens), 16 streams/GPU in closed loop, 64 rank-16 "
                "adapters over 800 classes")
    mode = args.loop
    m = binding.model_from_workload(w, dtype=0, max_frames=S, max_set=8)
    m.set_cover(w.tau)
    if args.whole_network_kernel is not None:
        m.set_small_batch_kernel(args.whole_network_kernel == "on")
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
    clip = clip_scores = None
    if mode == "sequence":
        # one eager clip, then all T steps of a clip are one recorded sequence reading a static clip buffer
        args.steps = (args.steps + T - 1) // T * T
        clip = frames_dev.clone()
        clip_scores = torch.zeros((T, S, K), device="cuda")
        clip_scores_host = torch.zeros((T, S, K)).pin_memory()
        r.reset()
        for t in range(T):
            r.step(clip[t])
        r.capture_sequence(clip, log_scores=clip_scores)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def loop(n, e2e, replay=True):
        if mode == "sequence" and replay:
            for _ in range(n // T):
                if e2e:
                    clip.copy_(frames_host, non_blocking=True)
                r.run_sequence()
                if e2e:
                    clip_scores_host.copy_(clip_scores, non_blocking=True)
            return
        for i in range(n):
            t = i % T
            if t == 0:
                r.reset()
            if mode == "graph" and replay:
                stage.copy_(frames_host[t] if e2e else frames_dev[t], non_blocking=True)
                sc, _ = r.step(stage) if t == 0 else r.step_graph()
            elif e2e:
                stage.copy_(frames_host[t], non_blocking=True)
                sc, _ = r.step(stage)
            else:
                sc, _ = r.step(frames_dev[t])
            if e2e:
                scores_host.copy_(sc, non_blocking=True)

    loop(max(args.warmup, 3) if mode != "sequence" else T, False)
    assert m.status() == 0
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else 0)
    if rank == 0:
        sampler.start()
    out_ms = []
    launches = 0
    walls = []
    for e2e in (False, True):
        if e2e:
            loop(2 if mode != "sequence" else T, True)
        barrier()
        count = lambda: m.launch_count() + (r.replayed_launches if mode in ("graph", "sequence") else 0)
        n0 = count()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        walls.append(time.time())
        e0.record(stream)
        loop(args.steps, e2e)
        e1.record(stream)
        barrier()
        walls.append(time.time())
        out_ms.append(e0.elapsed_time(e1))
        if not e2e:
            launches = count() - n0
    assert m.status() == 0
    # roofline pass: whole 30-step sequences, launched one by one (no replay) with events around each
    # launch site, for at least --roofline-seconds
    ms_step = out_ms[0] / args.steps
    n_seq = max(1, math.ceil(args.roofline_seconds * 1e3 / max(ms_step, 1e-3) / T))
    used_contexts = 0
    m.profile_enable(True)
    barrier()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    tw0 = time.time()
    p0.record(stream)
    for _ in range(n_seq):
        m.metrics_reset()
        loop(T, False, replay=False)
        _, chosen, _ = m.metrics_read()
        # the forwards of a sequence used the empty sets and what select chose at steps 0 .. T-2
        used_contexts += chosen - sum(len(s) for s in r.current_sets())
    p1.record(stream)
    barrier()
    tw1 = time.time()
    prof = m.profile_read()
    m.profile_enable(False)
    region_s = p0.elapsed_time(p1) * 1e-3
    sampler.stop()
    ms, ms_e2e = shard.max_over_ranks(out_ms, device="cuda")
    if rank == 0:
        peaks = measured_peaks()
        steps_r = n_seq * T
        # every chosen adapter has the same rank and placement: scale one adapter's LoRA work
        one = linear_flops(w.spec, w.adapters, [[0]])
        zero = linear_flops(w.spec, w.adapters, [[]])
        per_step = {k: zero[k] * S + (one[k] - zero[k]) * used_contexts / steps_r for k in zero}
        bts = hbm_bytes(w.spec, S, sum(len(a.class_ids) for a in w.adapters), len(w.adapters))
        clocks_r = sampler.window(tw0, tw1)
        roof, hbm_entries = roofline_block(prof, steps_r, per_step, bts, peaks, clocks_r, None, w.spec.layers, region_s)
        sample = 2 if args.workload == "streams" else 16
        fr = w.extra["stream_frames"]
        cv, cdt = oracle_frames_per_s(w, np.concatenate([fr[:1, t] for t in range(sample)]), [[] for _ in range(sample)]) \
            if args.cpu_sample > 0 and world == 1 else (None, 0.0)
        print(json.dumps({
            "metric": METRICS[args.workload], "value": world * S * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": max(args.warmup, 3), "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16", "data": "synthetic",
            "config": {"workload": what + ", sets chosen by Algorithm 2 on the device",
                       "streams_per_gpu": S,
                       "loop": {"host": "routing plan on the host (a device-to-host copy and a stream synchronisation per step)",
                                "device": "routing plan built on the device, no host synchronisation",
                                "graph": "routing plan built on the device; steps after a stream's first are CUDA-graph replays",
                                "sequence": "routing plan built on the device; a clip of 30 steps is one recorded sequence "
                                            "(one CUDA-graph launch per clip)"}[mode],
                       "l2": "one step's activations fit the 126 MB L2; no flush" if args.workload == "latency"
                             else "one step touches ~0.2 GB of activations; no flush"},
            "latency_us_per_step": 1e3 * ms / args.steps,
            "e2e": {"value": world * S * args.steps / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(stage.numel() * 2), "d2h_bytes_per_step": int(scores_host.numel() * 4)},
            "gpu_launches": int(launches),
            "clocks": sampler.window(walls[0], walls[1]),
            "clocks_roofline_pass": clocks_r,
            "roofline": roof, "roofline_hbm": hbm_entries,
            "kernel_ms_per_step": {k: v[0] / steps_r for k, v in prof.items()},
            "avg_active_adapters_per_frame": used_contexts / (steps_r * S),
            "cpu_baseline": None if cv is None else
                {"value": cv, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                 "sample": f"{sample} frames of one stream with the plain backbone, once ({cdt:.1f} s)"},
        }))
    m.close()
    if dist is not None:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=100)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="polymorph", choices=["polymorph", "reference"])
    ap.add_argument("--frames", type=int, default=256, help="frames per GPU per step")
    ap.add_argument("--cpu-sample", type=int, default=16, help="frames of the CPU-baseline sample (0 = skip)")
    ap.add_argument("--roofline-seconds", type=float, default=2.5,
                    help="the per-kernel pass runs at least this long (and at least --steps steps)")
    ap.add_argument("--sets-change", type=float, default=0.0, metavar="P",
                    help="batch workload: every step each frame redraws its adapter set with probability P, so the "
                         "routing plan is rebuilt and uploaded inside the timed region (0: the sets repeat and the "
                         "plan is reused, the headline configuration)")
    ap.add_argument("--device-sets", action="store_true",
                    help="batch workload: the set lists live on the device and the plan is built there "
                         "(pm_forward_device_sets)")
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
    ap.add_argument("--whole-network-kernel", default=None, choices=["on", "off"],
                    help="latency: one kernel per forward (a CTA per 16 token rows) or the layer-by-layer kernels; "
                         "default: the library's choice")
    ap.add_argument("--loop", default="graph", choices=["host", "device", "graph", "sequence"],
                    help="streams / latency: where the routing plan of a step is built and whether steps are "
                         "CUDA-graph replays (graph: one replay per step; sequence: the whole 30-step clip is one "
                         "recorded sequence, one graph launch per clip -- --steps is then rounded up to whole clips)")
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
        run_streams(args, rank, world, dist, local_rank)
        return

    w = wl.vit_base_batch(n_frames=args.frames, lora_last=args.lora_last)
    if args.branched and args.lora_last is None:
        raise SystemExit("--branched needs --lora-last N (adapters may not touch the shared trunk)")
    if args.branched and (args.sets_change > 0 or args.device_sets):
        raise SystemExit("--branched runs with fixed host sets only")
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

    # the adapter sets of every step: the workload's own (repeated), or a slowly changing sequence
    if args.sets_change > 0:
        seq = wl.changing_sets(w.sets(), 64, args.sets_change, len(w.adapters), "bench")
    else:
        seq = [(w.set_offsets, w.set_ids)]
    if args.device_sets:
        # pinned host copies: in the end-to-end pass a step's lists travel to the device like its frames
        seq_pinned = [(torch.from_numpy(o).pin_memory(), torch.from_numpy(i).pin_memory()) for o, i in seq]
        dev_lists = (torch.zeros(F + 1, dtype=torch.int32, device="cuda"),
                     torch.zeros(F * 3, dtype=torch.int32, device="cuda"))

    def sets_of(i):
        return seq[i % len(seq)]

    def step(i, frames=None):
        fr = frames_dev if frames is None else frames
        if args.branched:
            m.forward_branched(fr, w.set_offsets, w.set_ids, trunk, scores, base)
        elif args.device_sets:
            o, ids = seq_pinned[i % len(seq)]
            if args.sets_change > 0 or i == 0:
                dev_lists[0].copy_(o, non_blocking=True)
                dev_lists[1][:ids.numel()].copy_(ids, non_blocking=True)
            m.forward_device_sets(fr, dev_lists[0], dev_lists[1], scores, base)
        else:
            o, ids = sets_of(i)
            m.forward(fr, o, ids, scores, base)
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

    # ---- pass 1, the headline: exactly K steps, inputs resident in HBM ---------------------
    sampler = ClockSampler(local_rank if "CUDA_VISIBLE_DEVICES" not in os.environ else 0)
    if rank == 0:
        sampler.start()
    n0 = m.launch_count()
    plans0, plan_ms0 = m.plan_stats()
    barrier()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall0 = time.time()
    e0.record(stream)
    for i in range(args.steps):
        step(args.warmup + i)
    e1.record(stream)
    barrier()
    t_wall1 = time.time()
    ms = e0.elapsed_time(e1)
    launches = m.launch_count() - n0
    plans1, plan_ms1 = m.plan_stats()

    # ---- pass 2, the roofline: per-launch-site events, seconds long ------------------------
    steps_r = max(args.steps, math.ceil(args.roofline_seconds * 1e3 / max(ms / args.steps, 1e-3)))
    m.profile_enable(True)
    barrier()
    p0, p1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    t_wall2 = time.time()
    p0.record(stream)
    for i in range(steps_r):
        step(args.warmup + args.steps + i)
    p1.record(stream)
    barrier()
    t_wall3 = time.time()
    ms_profiled = p0.elapsed_time(p1)
    prof = m.profile_read()
    m.profile_enable(False)
    assert m.status() == 0, "device status word set during the timed region"

    # ---- pass 3, end to end: host frames in, host scores out, copies inside the timed region
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
    sampler.stop()

    ms, ms_e2e = shard.max_over_ranks([ms, ms_e2e], device="cuda")

    if rank == 0:
        peaks = measured_peaks()
        L = w.spec.layers
        if args.branched:
            branches = F + len(w.set_ids)
            rows = [F] * trunk + [branches] * (L - trunk)
            flops = linear_flops(w.spec, w.adapters, w.sets(), first_layer=trunk, rows_per_layer=rows)
        elif args.sets_change > 0:
            # mean over the sequence of set lists
            acc = None
            for o, ids in seq:
                sets = [list(map(int, ids[o[f]:o[f + 1]])) for f in range(F)]
                fl = linear_flops(w.spec, w.adapters, sets)
                acc = fl if acc is None else {k: acc[k] + fl[k] for k in fl}
            flops = {k: v / len(seq) for k, v in acc.items()}
        else:
            flops = linear_flops(w.spec, w.adapters, w.sets())
        bts = hbm_bytes(w.spec, F, sum(len(a.class_ids) for a in w.adapters), len(w.adapters))
        clocks_r = sampler.window(t_wall2, t_wall3)
        traffic = None if (args.branched or args.frames != 256) else dram_traffic("lora_gemm_pair_kernel")
        n_shrink_layers = L if args.lora_last is None else args.lora_last
        roof, hbm_entries = roofline_block(prof, steps_r, flops, bts, peaks, clocks_r, traffic, n_shrink_layers,
                                           ms_profiled * 1e-3)
        total_flops = sum(flops.values()) + 4 * w.spec.tokens ** 2 * w.spec.d * L * F      # + attention
        out = {
            "metric": METRICS["batch"], "value": world * F * args.steps / (ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "bf16",
            "data": "synthetic",
            "config": {"workload": "vit_base_batch: ViT-base 224x224 (197 tokens), %d frames/GPU/step, 32 rank-16 "
                                   "adapters over 800 classes, 1-3 active adapters per frame (60/30/10 %%), "
                                   "forward + Algorithm 2 select" % F,
                       "frames_per_gpu": F, "l2": "activations (~0.9 GB/step) exceed the 126 MB L2; no flush",
                       "lora_blocks": "all 12" if args.lora_last is None else "last %d" % args.lora_last,
                       "arrangement": ("branched: %d shared blocks, then %d branches for %d frames" %
                                       (trunk, F + len(w.set_ids), F)) if args.branched else "one stream per frame",
                       "sets": ("each frame redraws its set with probability %g per step" % args.sets_change)
                               if args.sets_change > 0 else "the same sets every step (routing plan reused)",
                       "plan": "built on the device from device-resident lists" if args.device_sets
                               else "built on the host"},
            "e2e": {"value": world * F * args.steps / (ms_e2e * 1e-3), "unit": UNIT,
                    "h2d_bytes_per_step": int(frames_host.numel() * 2) +
                                          (int(seq_pinned[0][0].numel() * 4 + F * 3 * 4) if args.device_sets else 0),
                    "d2h_bytes_per_step": int(scores_host.numel() * 4 + base_host.numel() * 4)},
            "gpu_launches": int(launches),
            "clocks": sampler.window(t_wall0, t_wall1),
            "clocks_roofline_pass": clocks_r,
            "whole_step_tflops": total_flops * args.steps / (ms * 1e-3) / 1e12,
            "roofline": roof,
            "roofline_hbm": hbm_entries,
            "kernel_ms_per_step": {k: v[0] / steps_r for k, v in prof.items()},
            "profiled_pass_ms_per_step": ms_profiled / steps_r,
            "host_plans_per_step": (plans1 - plans0) / args.steps,
            "host_plan_ms_per_step": (plan_ms1 - plan_ms0) / args.steps,
        }
        if args.cpu_sample > 0 and world == 1:
            n = min(args.cpu_sample, F)
            v, dt = oracle_frames_per_s(w, w.frames[:n], w.sets()[:n])
            out["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": host_threads(), "kind": "oracle",
                                   "sample": f"{n} of the {F} frames, once ({dt:.1f} s)"}
        else:
            out["cpu_baseline"] = None
        print(json.dumps(out))
    m.close()
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
