"""Closed-loop streaming (577-token ViT-base, 16 streams): forward -> Algorithm 2 on the device -> next
forward, free running.  Checked against the oracle by teacher forcing: the oracle is given the sets
the GPU actually used (scores within 1e-2) and the GPU's own base scores (selection bit-exact,
including the carried label state)."""
import numpy as np
import pytest

import workloads as wl
from oracle import polymorph_oracle as po


def check_device_metrics(out, n_streams):
    """AvgCoverage (Eq. 7) and SwitchPenalty (Eq. 8) counted on the device by pm_select against the
    oracle's definitions applied, per stream, to the sequence of sets Algorithm 2 chose."""
    chosen = out["chosen_sets"]
    per_stream = [[step[s] for step in chosen] for s in range(n_streams)]
    total = sum(len(seq) for seq in per_stream)
    assert out["avg_coverage"] == pytest.approx(sum(po.avg_coverage(seq) * len(seq) for seq in per_stream) / total)
    assert out["switch_penalty"] == sum(po.switch_penalty(seq) for seq in per_stream)


@pytest.mark.gpu
@pytest.mark.parametrize("context_copy,T", [(False, 30), (True, 5)])
def test_free_running_streams_teacher_forced(context_copy, T):
    """T = 30 is the full length of the streaming configuration (16 streams x 30 frames)."""
    import torch
    from paper_2507_14959_b200 import binding, streaming
    S = 16
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
    assert out["chosen_sets"][:-1] == used[1:]                      # what select chose is what the next forward used
    check_device_metrics(out, S)
    # forward: the oracle, given the sets the GPU used, reproduces sampled rows
    for (t, s) in [(1, 0), (T - 1, S - 1), (2, 7)]:
        off, ids = wl.sets_to_csr([used[t][s]])
        so, bo = po.forward(w.backbone, w.adapters, fr[s:s + 1, t], off, ids, w.spec.heads, w.spec.patch,
                            w.spec.ln_eps, w.spec.n_classes)
        assert np.abs(out["scores"][t, s] - so[0]).max() < 1e-2
        assert np.abs(base[t, s] - bo[0]).max() < 1e-2
    m.close()


@pytest.mark.gpu
def test_device_plan_and_graph_replay_match_host_plan():
    """The same closed loop three ways: plan on the host (pm_forward), plan on the device
    (pm_forward_device_sets), and the device-plan step replayed from CUDA graphs.  A row's result does
    not depend on where bucketing puts it; eager and replayed device-plan loops agree bit for bit."""
    import torch
    from paper_2507_14959_b200 import binding, streaming
    w = wl.deit_small_streams()
    S, T = 8, 6
    spec = w.spec
    fr = wl.make_stream_frames("device_plan_streams", spec, S, T)           # [S, T, 3, img, img]
    # a base-head bias that lets only a few labels per frame cross 0.5: small, non-empty sets
    bb = wl.make_backbone("device_plan_streams", spec, head_bias_mean=-0.9)
    w = wl.Workload("device_plan_streams", spec, bb, w.adapters, w.frames, w.set_offsets, w.set_ids)
    m = binding.model_from_workload(w, dtype=0, max_frames=S, max_set=16)
    m.set_cover(0.6)
    fd = torch.from_numpy(fr).cuda().to(torch.bfloat16)
    outs = [streaming.run(m, fd, spec.n_classes, len(w.adapters), 0.5, False, device_plan=dp, graph=gr)
            for dp, gr in ((False, False), (True, False), (True, True))]
    sizes = [len(x) for step in outs[0]["used_sets"][1:] for x in step]
    assert np.mean(sizes) > 0.5                                     # adapters really are in play
    # replaying the recorded step launches exactly the kernels of the eager device-plan step
    assert outs[2]["used_sets"] == outs[1]["used_sets"]
    np.testing.assert_array_equal(outs[2]["base"], outs[1]["base"])
    np.testing.assert_array_equal(outs[2]["scores"], outs[1]["scores"])
    # host plan against device plan: the first step (no adapters anywhere) runs the same frames through
    # slightly different arithmetic (the host plan skips the LoRA path and takes the LayerNorm statistics
    # from a kernel of their own, the device plan from the shrink), so scores agree to rounding only and
    # a label next to the threshold may flip; from then on each loop follows its own sets.  Every loop
    # must be consistent with Algorithm 2 applied to its own base scores.
    assert np.abs(outs[1]["base"][0] - outs[0]["base"][0]).max() < 5e-3
    contexts = [a.class_ids for a in w.adapters]
    accs = [a.acc for a in w.adapters]
    for o in outs:
        for st in range(S):
            Y_prev, S_prev = None, None
            for t in range(T - 1):
                Y = po.labels_from_scores(o["base"][t, st], 0.5)
                want = po.detect_contexts(Y, Y_prev, contexts, accs, 0.6, S_prev, False)
                assert want == o["used_sets"][t + 1][st], (st, t)
                Y_prev, S_prev = Y, want
    # the device-plan loop against the oracle, teacher-forced with the sets that loop used
    for (t, st) in [(2, 1), (T - 1, S - 1)]:
        off, ids = wl.sets_to_csr([outs[1]["used_sets"][t][st]])
        so, bo = po.forward(w.backbone, w.adapters, fr[st:st + 1, t], off, ids, spec.heads, spec.patch,
                            spec.ln_eps, spec.n_classes)
        assert np.abs(outs[1]["scores"][t, st] - so[0]).max() < 1e-2
        assert np.abs(outs[1]["base"][t, st] - bo[0]).max() < 1e-2
    for o in outs:
        check_device_metrics(o, S)
    # the whole clip as ONE recorded sequence (T steps in a single graph launch): same bits, same counters
    r = outs[1]["runner"]
    clip = fd.transpose(0, 1).contiguous()                          # [T, S, 3, img, img]
    log_b = torch.zeros((T, S, spec.n_classes), device="cuda")
    log_s = torch.zeros_like(log_b)
    r.capture_sequence(clip, log_b, log_s)
    for _ in range(2):                                              # a replay leaves no state behind
        log_b.fill_(-1.0)
        m.metrics_reset()
        r.run_sequence()
        n, contexts, switches = m.metrics_read()
        np.testing.assert_array_equal(log_b.cpu().numpy(), outs[1]["base"])
        np.testing.assert_array_equal(log_s.cpu().numpy(), outs[1]["scores"])
        assert r.current_sets() == outs[1]["chosen_sets"][-1]
        assert n == S * T and contexts / n == pytest.approx(outs[1]["avg_coverage"])
        assert switches == outs[1]["switch_penalty"]
    assert m.status() == 0
    m.close()


@pytest.mark.gpu
@pytest.mark.parametrize("dtype", [0, 1])
def test_device_plan_reports_bad_lists(dtype):
    import torch
    from paper_2507_14959_b200 import binding
    w = wl.deit_tiny_2frames()
    m = binding.model_from_workload(w, dtype=dtype, max_frames=2, max_set=2)
    fd = torch.from_numpy(w.frames).cuda()
    fd = fd.to(torch.bfloat16) if dtype == 0 else fd
    K = w.spec.n_classes
    sc, bs = torch.zeros((2, K), device="cuda"), torch.zeros((2, K), device="cuda")
    ref_s, ref_b = torch.zeros((2, K), device="cuda"), torch.zeros((2, K), device="cuda")
    off = torch.tensor([0, 1, 3], dtype=torch.int32, device="cuda")
    m.forward_device_sets(fd, off, torch.tensor([0, 1, 3], dtype=torch.int32, device="cuda"), ref_s, ref_b)
    assert m.status() == 0
    so, bo = po.forward(w.backbone, w.adapters, w.frames, w.set_offsets, w.set_ids, w.spec.heads, w.spec.patch,
                        w.spec.ln_eps, K)
    tol = 1e-2 if dtype == 0 else 1e-4
    assert np.abs(ref_s.cpu().numpy() - so).max() < tol and np.abs(ref_b.cpu().numpy() - bo).max() < tol
    # id 9 is out of range, id 3 repeated: both are skipped and the status word says so
    m.forward_device_sets(fd, torch.tensor([0, 2, 5], dtype=torch.int32, device="cuda"),
                          torch.tensor([0, 9, 3, 1, 3], dtype=torch.int32, device="cuda"), sc, bs)
    assert m.status() == binding.PM_ERR_ARG
    np.testing.assert_array_equal(sc.cpu().numpy(), ref_s.cpu().numpy())
    # three ids where max_set is 2: the two lowest are kept
    m.forward_device_sets(fd, torch.tensor([0, 1, 4], dtype=torch.int32, device="cuda"),
                          torch.tensor([0, 3, 2, 1], dtype=torch.int32, device="cuda"), sc, bs)
    assert m.status() == binding.PM_ERR_CAPACITY
    m.close()


@pytest.mark.gpu
def test_single_stream_latency_shape_teacher_forced():
    """DeiT-tiny, one stream, query/value adapters on the last two blocks (Sec. 4, Table 2 shape), closed
    loop as CUDA-graph replays: the oracle, given the sets the GPU used, reproduces every step."""
    import torch
    from paper_2507_14959_b200 import binding, streaming
    T = 5
    w = wl.deit_tiny_stream(n_steps=T, n_streams=1)
    m = binding.model_from_workload(w, dtype=0, max_frames=1, max_set=8)
    m.set_cover(w.tau)
    fr = w.extra["stream_frames"]
    fd = torch.from_numpy(fr).cuda().to(torch.bfloat16)
    out = streaming.run(m, fd, w.spec.n_classes, len(w.adapters), 0.5, False, device_plan=True, graph=True)
    used, base = out["used_sets"], out["base"]
    contexts = [a.class_ids for a in w.adapters]
    accs = [a.acc for a in w.adapters]
    Y_prev, S_prev = None, None
    for t in range(T):
        off, ids = wl.sets_to_csr([used[t][0]])
        so, bo = po.forward(w.backbone, w.adapters, fr[0:1, t], off, ids, w.spec.heads, w.spec.patch,
                            w.spec.ln_eps, w.spec.n_classes)
        assert np.abs(out["scores"][t, 0] - so[0]).max() < 1e-2
        assert np.abs(base[t, 0] - bo[0]).max() < 1e-2
        if t + 1 < T:
            Y = po.labels_from_scores(base[t, 0], 0.5)
            want = po.detect_contexts(Y, Y_prev, contexts, accs, w.tau, S_prev, False)
            assert want == used[t + 1][0], t
            Y_prev, S_prev = Y, want
    assert sum(len(s[0]) for s in used[1:]) > 0
    m.close()
