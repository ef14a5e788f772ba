"""Closed-loop streaming driver: for every time step, one pm_forward over the current frame of each
stream with the adapter sets chosen at the previous step, then pm_select (Algorithm 2) on the base
scores to choose the sets for the next frame.  The scores never leave the device; the id lists
produced by pm_select are handed straight back to pm_forward.

Also counts the two stream-level metrics of the paper on the sets that were actually used:
AvgCoverage (Eq. 7, mean number of active contexts per frame) and SwitchPenalty (Eq. 8, number of
steps at which a stream's set changed).
"""
from __future__ import annotations

import numpy as np


class StreamRunner:
    """Owns the per-stream device state (previous label bit sets, two CSR buffers that alternate
    between "sets of this step" and "sets for the next step")."""

    def __init__(self, model, n_streams, n_classes, n_adapters, score_thr=0.5, context_copy=False):
        import torch
        self.model = model
        self.S = n_streams
        self.K = n_classes
        self.score_thr = float(score_thr)
        self.context_copy = bool(context_copy)
        dev = "cuda"
        self.scores = torch.zeros((n_streams, n_classes), device=dev)
        self.base = torch.zeros((n_streams, n_classes), device=dev)
        self.labels = torch.zeros((n_streams, (n_classes + 31) // 32), dtype=torch.int32, device=dev)
        self.csr = [(torch.zeros(n_streams + 1, dtype=torch.int32, device=dev),
                     torch.zeros(max(1, n_streams * n_adapters), dtype=torch.int32, device=dev)) for _ in range(2)]
        self.t = 0

    def reset(self):
        """Next step is the first frame of every stream: empty sets, no previous labels."""
        for off, _ in self.csr:
            off.zero_()
        self.t = 0

    def step(self, frames):
        """frames: device tensor [n_streams, 3, img, img].  Runs the forward with the current sets and
        selects the next ones.  Returns (scores, base_scores) device tensors (overwritten next step)."""
        cur, nxt = self.csr[self.t % 2], self.csr[(self.t + 1) % 2]
        self.model.forward(frames, cur[0], cur[1], self.scores, self.base)
        self.model.select(self.base, self.score_thr, self.context_copy, self.t > 0, self.labels,
                          cur[0], cur[1], nxt[0], nxt[1])
        self.t += 1
        return self.scores, self.base

    def current_sets(self):
        """The sets the next step will use, as host lists (synchronises)."""
        off, ids = self.csr[self.t % 2]
        o = off.cpu().numpy()
        i = ids.cpu().numpy()
        return [list(map(int, i[o[f]:o[f + 1]])) for f in range(self.S)]


def avg_coverage(sets_per_step):
    """Eq. 7 over all streams: mean |S_t| per frame."""
    n = sum(len(step) for step in sets_per_step)
    return sum(len(s) for step in sets_per_step for s in step) / max(n, 1)


def switch_penalty(sets_per_step):
    """Eq. 8 summed over streams: number of (stream, t >= 1) with S_t != S_{t-1}."""
    total = 0
    for t in range(1, len(sets_per_step)):
        total += sum(1 for a, b in zip(sets_per_step[t - 1], sets_per_step[t]) if sorted(a) != sorted(b))
    return total


def run(model, frames_seq, n_classes, n_adapters, score_thr=0.5, context_copy=False, record=True):
    """frames_seq: device tensor [n_streams, n_steps, 3, img, img].  Free-running loop over all steps.
    Returns {"used_sets": per step the sets the forward used, "base": [n_steps, S, K] numpy,
    "scores": same, "avg_coverage", "switch_penalty"} (records only if `record`)."""
    S, T = int(frames_seq.shape[0]), int(frames_seq.shape[1])
    r = StreamRunner(model, S, n_classes, n_adapters, score_thr, context_copy)
    r.reset()
    used, base_log, score_log = [], [], []
    for t in range(T):
        if record:
            used.append(r.current_sets())
        scores, base = r.step(frames_seq[:, t].contiguous())
        if record:
            base_log.append(base.cpu().numpy().copy())
            score_log.append(scores.cpu().numpy().copy())
    if model.status() != 0:
        raise RuntimeError("device status word set during the streaming loop")
    out = {"runner": r}
    if record:
        out.update(used_sets=used, base=np.stack(base_log), scores=np.stack(score_log),
                   avg_coverage=avg_coverage(used), switch_penalty=switch_penalty(used))
    return out
