"""Closed-loop streaming (577-token ViT-base, 16 streams): forward -> Algorithm 2 on the device -> next
forward, free running.  Checked against the oracle by teacher forcing: the oracle is given the sets
the GPU actually used (scores within 1e-2) and the GPU's own base scores (selection bit-exact,
including the carried label state)."""
import numpy as np
import pytest

import workloads as wl
from oracle import polymorph_oracle as po


def test_stream_metrics_match_eq7_eq8():
    from paper_2507_14959_b200 import streaming
    # 2 streams, 4 steps
    steps = [[[0], [1, 2]], [[0], [1, 2]], [[0, 3], [2]], [[0, 3], []]]
    per_stream = [[s[i] for s in steps] for i in range(2)]
    assert streaming.avg_coverage(steps) == pytest.approx(
        sum(po.avg_coverage(seq) * len(seq) for seq in per_stream) / 8)
    assert streaming.switch_penalty(steps) == sum(po.switch_penalty(seq) for seq in per_stream)


@pytest.mark.gpu
@pytest.mark.parametrize("context_copy", [False, True])
def test_free_running_streams_teacher_forced(context_copy):
    import torch
    from paper_2507_14959_b200 import binding, streaming
    S, T = 16, 5
    w = wl.vit_base_384_streams(n_streams=S, n_steps=T)
    m = binding.model_from_workload(w, dtype=0, max_frames=S, max_set=8)
    m.set_cover(w.tau)
    fr = w.extra["stream_frames"]                                   # [S, T, 3, 384, 384]
    fd = torch.from_numpy(fr).cuda().to(torch.bfloat16)
    out = streaming.run(m, fd, w.spec.n_classes, len(w.adapters), 0.5, context_copy)
    used, base = out["used_sets"], out["base"]
    assert all(len(s) == 0 for s in used[0])                        # first frame: plain backbone
    contexts = [a.class_ids for a in w.adapters]
    accs = [a.acc for a in w.adapters]
    # selection: the sets used at t+1 are Algorithm 2 applied to the GPU's base scores of step t
    for s in range(S):
        Y_prev, S_prev = None, None
        for t in range(T - 1):
            Y = po.labels_from_scores(base[t, s], 0.5)
            want = po.detect_contexts(Y, Y_prev, contexts, accs, w.tau, S_prev, context_copy)
            assert want == used[t + 1][s], (s, t)
            Y_prev, S_prev = Y, want
    sizes = [len(x) for step in used[1:] for x in step]
    assert 0 < np.mean(sizes) <= 8
    # forward: the oracle, given the sets the GPU used, reproduces sampled rows
    for (t, s) in [(1, 0), (T - 1, S - 1), (2, 7)]:
        off, ids = wl.sets_to_csr([used[t][s]])
        so, bo = po.forward(w.backbone, w.adapters, fr[s:s + 1, t], off, ids, w.spec.heads, w.spec.patch,
                            w.spec.ln_eps, w.spec.n_classes)
        assert np.abs(out["scores"][t, s] - so[0]).max() < 1e-2
        assert np.abs(base[t, s] - bo[0]).max() < 1e-2
    m.close()
