"""pm_select_static -- the selection entry point for callers that may not allocate device memory
(no-allocation control loops, plug-ins inside another framework's memory pool): its scratch lives
in a fixed array inside the library.  It must return exactly what pm_select returns on the same
inputs, on consecutive calls that reuse the shared array.  This file is collected last on purpose,
so a stop-at-first-failure run has already been through every other test."""
import numpy as np
import pytest

import workloads as wl

pytestmark = pytest.mark.gpu

TAU = 0.6


def cover_tables(ctxs, accs, n_classes, tau):
    """first[k] and provider[k, words] as the header describes them (fewest classes first, then id)."""
    n_ad = len(ctxs)
    words = max(1, (n_ad + 63) // 64)
    first = np.full(n_classes, -1, np.int32)
    provider = np.zeros((n_classes, words), np.uint64)
    for a in sorted(range(n_ad), key=lambda a: (len(ctxs[a]), a)):
        for j, k in enumerate(ctxs[a]):
            if accs[a][j] >= tau:
                if first[k] < 0:
                    first[k] = a
                provider[k, a // 64] |= np.uint64(1) << np.uint64(a % 64)
    return first, provider


def handle_model(ctxs, accs, n_classes, max_frames):
    from paper_2507_14959_b200 import binding
    spec = wl.ModelSpec(img=32, d=64, heads=1, mlp=64, n_classes=n_classes, layers=1)
    m = binding.Model(img=32, d=64, layers=1, heads=1, mlp=64, n_classes=n_classes,
                      backbone=wl.make_backbone("no_alloc", spec), max_adapters=len(ctxs), max_rank=16,
                      max_set=4, max_frames=max_frames)
    for a, (c, ac) in enumerate(zip(ctxs, accs)):
        m.register_adapter(a, rank=1, scale=1.0, A=[None] * 4, B=[None] * 4, class_ids=c,
                           head_w=np.zeros((64, len(c)), np.float32), head_b=np.zeros(len(c), np.float32), acc=ac)
    m.set_cover(TAU)
    return m


def draw_scores(g, F, K):
    s = np.full((F, K), 0.1, np.float32)
    for f in range(F):
        s[f, g.choice(K, size=int(g.integers(0, 5)), replace=False)] = 0.9
    return s


@pytest.mark.parametrize("n_ctx,n_labels,max_size,context_copy", [(70, 200, 9, True), (12, 40, 6, False)])
def test_static_scratch_select_matches_pm_select_on_two_calls(n_ctx, n_labels, max_size, context_copy):
    import torch
    from paper_2507_14959_b200 import binding
    ctxs, accs = wl.random_cover_table(11, n_ctx, n_labels, max_size, True)
    keep = [i for i, c in enumerate(ctxs) if len(c)]
    ctxs, accs = [ctxs[i] for i in keep], [accs[i] for i in keep]
    F, n_ad = 53, len(ctxs)
    m = handle_model(ctxs, accs, n_labels, F)
    first, provider = cover_tables(ctxs, accs, n_labels, TAU)
    first_d, prov_d = torch.from_numpy(first).cuda(), torch.from_numpy(provider.view(np.int64)).cuda()
    g = wl.rng_for("no_alloc_scores", n_ctx)
    nw = (n_labels + 31) // 32

    def state():
        return dict(labels=torch.zeros((F, nw), dtype=torch.int32, device="cuda"),
                    bufs=[(torch.zeros(F + 1, dtype=torch.int32, device="cuda"),
                           torch.full((F * n_ad,), -1, dtype=torch.int32, device="cuda")) for _ in range(2)])
    ref, new = state(), state()
    status = torch.full((1,), 77, dtype=torch.int32, device="cuda")     # the call must clear it
    scores0 = draw_scores(g, F, n_labels)
    scores1 = scores0.copy()
    changed = g.random(F) < 0.6
    scores1[changed] = draw_scores(g, int(changed.sum()), n_labels)
    for step, sc in enumerate([scores0, scores1]):        # two calls in a row share the static array
        sd = torch.from_numpy(sc).cuda()
        for st, static in ((ref, False), (new, True)):
            prev, nxt = st["bufs"][(step + 1) % 2], st["bufs"][step % 2]
            if static:
                binding.select_static(sd, n_ad, 0.5, context_copy, step > 0, st["labels"], prev[0], prev[1],
                                      first_d, prov_d, nxt[0], nxt[1], status_out=status)
            else:
                m.select(sd, 0.5, context_copy, step > 0, st["labels"], prev[0], prev[1], nxt[0], nxt[1])
        assert m.status() == 0
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        a, b = ref["bufs"][step % 2], new["bufs"][step % 2]
        assert torch.equal(a[0], b[0])
        n = int(a[0][-1].item())
        assert n > 0 and torch.equal(a[1][:n], b[1][:n])
        assert torch.equal(ref["labels"], new["labels"])
    m.close()


def test_static_scratch_select_rejects_sizes_beyond_its_array():
    import torch
    from paper_2507_14959_b200 import binding
    K = 8
    scores = torch.zeros((4097, K), device="cuda")
    first = torch.zeros(K, dtype=torch.int32, device="cuda")
    prov = torch.zeros((K, 5), dtype=torch.int64, device="cuda")
    off = torch.full((4098,), -5, dtype=torch.int32, device="cuda")
    ids = torch.zeros(16, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.PolymorphError) as e:          # more frames than the array holds
        binding.select_static(scores, 4, 0.5, False, False, None, None, None, first, prov, off, ids)
    assert e.value.code == binding.PM_ERR_CAPACITY
    with pytest.raises(binding.PolymorphError) as e:          # more adapters than the array holds
        binding.select_static(scores[:4], 257, 0.5, False, False, None, None, None, first, prov, off, ids)
    assert e.value.code == binding.PM_ERR_CAPACITY
    torch.cuda.synchronize()
    assert int(off.min().item()) == -5                        # nothing ran
    # capacity overflow of the id list is reported through status_out
    first[:] = torch.arange(K, dtype=torch.int32)
    prov[:, 0] = 1 << torch.arange(K, dtype=torch.int64)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    binding.select_static(torch.ones((2, K), device="cuda"), K, 0.5, False, False, None, None, None, first,
                          prov[:, :1].contiguous(), off, ids[:5], status_out=status)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.PM_ERR_CAPACITY
    assert off[:3].tolist() == [0, 8, 16]
