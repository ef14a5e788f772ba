"""Closed-loop streaming driver: for every time step, one pm_forward over the current frame of each
stream with the adapter sets chosen at the previous step, then pm_select (Algorithm 2) on the base
scores to choose the sets for the next frame.  The scores never leave the device; the id lists
produced by pm_select are handed straight back to the forward.  With ``device_plan`` (the default)
the forward is pm_forward_device_sets, which also builds its routing plan on the device, so a step
involves no host synchronisation at all and can be recorded once as a CUDA graph and replayed
(``capture`` / ``step_graph``); without it pm_forward copies the lists to the host to plan there.

The two stream-level metrics of the paper -- AvgCoverage (Eq. 7, mean number of active contexts per
frame) and SwitchPenalty (Eq. 8, number of steps at which a stream's set changed) -- are counted on
the device by pm_select over the sets it chooses (pm_metrics_read); nothing here touches the id lists
on the host unless ``record`` asks for them.
"""
from __future__ import annotations

import numpy as np


class StreamRunner:
    """Owns the per-stream device state (previous label bit sets, two CSR buffers that alternate
    between "sets of this step" and "sets for the next step")."""

    def __init__(self, model, n_streams, n_classes, n_adapters, score_thr=0.5, context_copy=False,
                 device_plan=True):
        import torch
        self.model = model
        self.device_plan = bool(device_plan)
        self.graphs = None
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
        self._enqueue(frames, self.t % 2, self.t > 0)
        self.t += 1
        return self.scores, self.base

    def _enqueue(self, frames, parity, has_prev):
        cur, nxt = self.csr[parity], self.csr[1 - parity]
        fwd = self.model.forward_device_sets if self.device_plan else self.model.forward
        fwd(frames, cur[0], cur[1], self.scores, self.base)
        self.model.select(self.base, self.score_thr, self.context_copy, has_prev, self.labels,
                          cur[0], cur[1], nxt[0], nxt[1])

    def capture(self, frames_static):
        """Records the step (forward from `frames_static`, then select) as two CUDA graphs, one per
        parity of the alternating list buffers.  Needs device_plan and one eager step before it (so
        that every kernel has been set up).  Afterwards: write the next frames into `frames_static`,
        call step_graph()."""
        import torch
        if not self.device_plan:
            raise ValueError("capture needs device_plan (the host planner synchronises the stream)")
        self.static_frames = frames_static
        self.graphs, self.graph_launches = [], []
        for parity in (0, 1):
            g = torch.cuda.CUDAGraph()
            n0 = self.model.launch_count()
            with torch.cuda.graph(g):
                self._enqueue(frames_static, parity, True)
            self.graphs.append(g)
            self.graph_launches.append(self.model.launch_count() - n0)
        self.replayed_launches = 0

    def step_graph(self):
        """Replays the recorded step on the frames currently in the static buffer (not the first
        step of a stream: that one has no previous labels and runs through step())."""
        if self.t == 0:
            raise ValueError("the first step of a stream runs through step()")
        p = self.t % 2
        self.graphs[p].replay()
        self.replayed_launches += self.graph_launches[p]
        self.t += 1
        return self.scores, self.base

    def capture_sequence(self, frames_seq, log_base=None, log_scores=None):
        """Records the closed loop over a whole clip -- frames_seq: device tensor [T, n_streams, 3, img,
        img], kept and re-read on every replay -- as ONE CUDA graph: empty sets for the first frame, then
        T times forward -> select, each step reading the lists the step before wrote.  log_base /
        log_scores ([T, n_streams, n_classes] device tensors, optional) receive every step's scores
        inside the graph.  Needs device_plan and one eager pass over a clip before it.  Replay with
        run_sequence(); to process another clip, copy its frames into frames_seq first."""
        import torch
        if not self.device_plan:
            raise ValueError("capture_sequence needs device_plan (the host planner synchronises the stream)")
        T = int(frames_seq.shape[0])
        g = torch.cuda.CUDAGraph()
        n0 = self.model.launch_count()
        with torch.cuda.graph(g):
            for off, _ in self.csr:
                off.zero_()
            for t in range(T):
                self._enqueue(frames_seq[t], t % 2, t > 0)
                if log_base is not None:
                    log_base[t].copy_(self.base)
                if log_scores is not None:
                    log_scores[t].copy_(self.scores)
        self.seq_graph, self.seq_steps = g, T
        self.seq_launches = self.model.launch_count() - n0
        self.replayed_launches = getattr(self, "replayed_launches", 0)

    def run_sequence(self):
        """Replays the recorded clip (capture_sequence): one graph launch for all its steps."""
        self.seq_graph.replay()
        self.replayed_launches += self.seq_launches
        self.t = self.seq_steps
        return self.scores, self.base

    def current_sets(self):
        """The sets the next step will use, as host lists (synchronises)."""
        off, ids = self.csr[self.t % 2]
        o = off.cpu().numpy()
        i = ids.cpu().numpy()
        return [list(map(int, i[o[f]:o[f + 1]])) for f in range(self.S)]


def run(model, frames_seq, n_classes, n_adapters, score_thr=0.5, context_copy=False, record=True,
        device_plan=True, graph=False):
    """frames_seq: device tensor [n_streams, n_steps, 3, img, img].  Free-running loop over all steps
    (graph: steps after the first are CUDA-graph replays).  Returns {"used_sets": per step the sets the forward used, "base": [n_steps, S, K] numpy,
    "chosen_sets": per step the sets pm_select chose for the next frame, "scores": same} (only if
    `record`; recording copies the lists to the host every step) and always "avg_coverage" (Eq. 7) and
    "switch_penalty" (Eq. 8, summed over streams) of the chosen sets, read once from the device counters
    after the last step."""
    S, T = int(frames_seq.shape[0]), int(frames_seq.shape[1])
    r = StreamRunner(model, S, n_classes, n_adapters, score_thr, context_copy, device_plan)
    r.reset()
    model.metrics_reset()
    used, chosen, base_log, score_log = [], [], [], []
    static = frames_seq[:, 0].contiguous() if graph else None
    for t in range(T):
        if record:
            used.append(r.current_sets())
        if graph and t > 0:
            if r.graphs is None:
                r.capture(static)
            static.copy_(frames_seq[:, t])
            scores, base = r.step_graph()
        else:
            scores, base = r.step(frames_seq[:, t].contiguous())
        if record:
            chosen.append(r.current_sets())
            base_log.append(base.cpu().numpy().copy())
            score_log.append(scores.cpu().numpy().copy())
    if model.status() != 0:
        raise RuntimeError("device status word set during the streaming loop")
    n, contexts, switches = model.metrics_read()
    out = {"runner": r, "avg_coverage": contexts / max(n, 1), "switch_penalty": switches}
    if record:
        out.update(used_sets=used, chosen_sets=chosen, base=np.stack(base_log), scores=np.stack(score_log))
    return out
