"""pm_select (Algorithm 2 on the device) against the oracle's literal Algorithm 2: bit-exact adapter
sets over several chained time steps, on disjoint and overlapping class->adapter tables."""
import numpy as np
import pytest

import workloads as wl
from oracle import polymorph_oracle as po

pytestmark = pytest.mark.gpu


def small_model(contexts, accs, n_classes, max_frames):
    from paper_2507_14959_b200 import binding
    spec = wl.ModelSpec(img=32, d=64, heads=1, mlp=64, n_classes=n_classes, layers=1)
    bb = wl.make_backbone("select_gpu", spec)
    m = binding.Model(img=32, d=64, layers=1, heads=1, mlp=64, n_classes=n_classes, backbone=bb,
                      max_adapters=len(contexts), max_rank=16, max_set=4, max_frames=max_frames)
    for a, (c, ac) in enumerate(zip(contexts, accs)):
        m.register_adapter(a, rank=1, scale=1.0, A=[None] * 4, B=[None] * 4, class_ids=c,
                           head_w=np.zeros((64, len(c)), np.float32), head_b=np.zeros(len(c), np.float32),
                           acc=ac)
    return m


@pytest.mark.parametrize("n_ctx,n_labels,max_size,overlap,seed", [
    (8, 16, 4, False, 0), (12, 40, 6, True, 1), (70, 200, 9, True, 2), (64, 800, 25, True, 3),
    (5, 33, 3, False, 4)])
@pytest.mark.parametrize("context_copy", [False, True])
def test_select_chained_steps(n_ctx, n_labels, max_size, overlap, seed, context_copy):
    import torch
    ctxs, accs = wl.random_cover_table(seed, n_ctx, n_labels, max_size, overlap)
    keep = [i for i, c in enumerate(ctxs) if len(c)]
    ctxs, accs = [ctxs[i] for i in keep], [accs[i] for i in keep]
    F = 37
    m = small_model(ctxs, accs, n_labels, F)
    tau = 0.6
    m.set_cover(tau)
    g = wl.rng_for("select_scores", seed, context_copy)
    nw = (n_labels + 31) // 32
    labels = torch.zeros((F, nw), dtype=torch.int32, device="cuda")
    cap = F * len(ctxs)
    bufs = [(torch.zeros(F + 1, dtype=torch.int32, device="cuda"),
             torch.full((cap,), -1, dtype=torch.int32, device="cuda")) for _ in range(2)]
    Y_prev = [None] * F
    S_prev = [None] * F
    cur = None
    for step in range(5):
        scores = np.full((F, n_labels), 0.1, dtype=np.float32)
        for f in range(F):
            if step > 0 and g.random() < 0.5:
                scores[f] = last[f]                     # unchanged frame: Y_t = Y_{t-1}
                continue
            on = g.choice(n_labels, size=int(g.integers(0, 5)), replace=False)
            scores[f, on] = 0.9
            scores[f, g.integers(0, n_labels)] = 0.5    # exactly at the threshold: not a label
        last = scores
        want = []
        for f in range(F):
            Y = po.labels_from_scores(scores[f], 0.5)
            want.append(po.detect_contexts(Y, Y_prev[f], ctxs, accs, tau, S_prev[f], context_copy))
            Y_prev[f], S_prev[f] = Y, want[-1]
        nxt = bufs[step % 2]
        m.select(torch.from_numpy(scores).cuda(), 0.5, context_copy, step > 0, labels,
                 None if cur is None else cur[0], None if cur is None else cur[1], nxt[0], nxt[1])
        assert m.status() == 0
        off, ids = wl.sets_to_csr(want)
        np.testing.assert_array_equal(nxt[0].cpu().numpy(), off)
        np.testing.assert_array_equal(nxt[1].cpu().numpy()[:len(ids)], ids)
        # the label bit sets written back are Y_t
        lab = labels.cpu().numpy().view(np.uint32)
        for f in range(F):
            bits = {k for k in range(n_labels) if (lab[f, k // 32] >> (k % 32)) & 1}
            assert bits == Y_prev[f]
        cur = nxt
    m.close()


def test_select_capacity_overflow_sets_status():
    import torch
    from paper_2507_14959_b200 import binding
    ctxs = [np.array([k], np.int32) for k in range(6)]
    accs = [np.ones(1, np.float32) for _ in range(6)]
    m = small_model(ctxs, accs, 6, 2)
    m.set_cover(0.5)
    scores = torch.ones((2, 6), device="cuda")
    noff = torch.zeros(3, dtype=torch.int32, device="cuda")
    nids = torch.zeros(7, dtype=torch.int32, device="cuda")       # 12 needed
    m.select(scores, 0.5, False, False, None, None, None, noff, nids)
    assert m.status() == binding.PM_ERR_CAPACITY
    assert m.status() == 0                                         # cleared after reading
    np.testing.assert_array_equal(noff.cpu().numpy(), [0, 6, 12])
    m.close()


def test_select_needs_cover_table():
    import torch
    from paper_2507_14959_b200 import binding
    ctxs = [np.array([0, 1], np.int32)]
    m = small_model(ctxs, [np.ones(2, np.float32)], 4, 1)
    with pytest.raises(binding.PolymorphError) as e:
        m.select(torch.zeros((1, 4), device="cuda"), 0.5, False, False, None, None, None,
                 torch.zeros(2, dtype=torch.int32, device="cuda"), torch.zeros(4, dtype=torch.int32, device="cuda"))
    assert e.value.code == binding.PM_ERR_STATE
    m.close()
