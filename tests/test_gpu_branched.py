"""GPU parity of pm_forward_branched (shared trunk, then one branch per active adapter: Fig. 2b,
Fig. 5b) against the oracle's branch reading, which runs every branch as a complete forward of its
own.  Scores: abs 1e-2 (bf16 build) / 1e-4 (fp32 debug build)."""
import numpy as np
import pytest

import workloads as wl
from oracle import polymorph_oracle as po

pytestmark = pytest.mark.gpu

SCORE_TOL = {0: 1e-2, 1: 1e-4}


def frames_to_dev(frames, dtype):
    import torch
    t = torch.from_numpy(np.ascontiguousarray(frames, dtype=np.float32)).cuda()
    return (t.to(torch.bfloat16) if dtype == 0 else t).contiguous()


def tiny_branch_workload(n_frames, sets, last=2, ab_std=0.05):
    """DeiT-tiny with four rank-4 adapters on the last `last` blocks only; class lists overlap
    (adapter a lists 6a .. 6a+9) so that the merge of branch outputs matters."""
    name = "deit_tiny_branched"
    spec = wl.tiny_spec(32)
    bb = wl.make_backbone(name, spec)
    ads = [wl.make_adapter(name, spec, a, 4, np.arange(6 * a, 6 * a + 10),
                           layers=range(spec.layers - last, spec.layers), ab_std=ab_std) for a in range(4)]
    off, ids = wl.sets_to_csr(sets)
    return wl.Workload(name, spec, bb, ads, wl.make_frames(name, spec, n_frames), off, ids)


def run_branched(m, w, dtype, trunk, with_base=True, frames=None, offsets=None, ids=None):
    import torch
    frames = w.frames if frames is None else frames
    offsets = w.set_offsets if offsets is None else offsets
    ids = w.set_ids if ids is None else ids
    F, K = frames.shape[0], w.spec.n_classes
    scores = torch.full((F, K), float("nan"), device="cuda")
    base = torch.full((F, K), float("nan"), device="cuda") if with_base else None
    m.forward_branched(frames_to_dev(frames, dtype), offsets, ids, trunk, scores, base)
    assert m.status() == 0
    s = scores.cpu().numpy().astype(np.float64)
    return (s, base.cpu().numpy().astype(np.float64)) if with_base else (s, None)


def oracle_branched(w, rows=None):
    rows = range(w.frames.shape[0]) if rows is None else rows
    sets = [list(w.set_ids[w.set_offsets[f]:w.set_offsets[f + 1]]) for f in rows]
    off, ids = wl.sets_to_csr(sets)
    return po.forward_branched(w.backbone, w.adapters, w.frames[list(rows)], off, ids, w.spec.heads,
                               w.spec.patch, w.spec.ln_eps, w.spec.n_classes)


@pytest.mark.parametrize("dtype", [1, 0])
def test_branched_deit_tiny(dtype):
    from paper_2507_14959_b200 import binding
    sets = [[0], [1, 3], [], [2, 0, 1]]
    w = tiny_branch_workload(4, sets)
    L = w.spec.layers
    m = binding.model_from_workload(w, dtype=dtype, max_frames=4 + 6)
    so, bo = oracle_branched(w)
    # the two readings of the paper differ on frames with several adapters by more than the tolerance,
    # so this parity separates them
    s1, b1 = po.forward(w.backbone, w.adapters, w.frames, w.set_offsets, w.set_ids, w.spec.heads,
                        w.spec.patch, w.spec.ln_eps, w.spec.n_classes)
    assert max(np.abs(s1 - so).max(), np.abs(b1 - bo).max()) > 3 * SCORE_TOL[0]
    for trunk in (L - 2, 0, 5):                 # any split at or before the first adapted block is the same function
        s, b = run_branched(m, w, dtype, trunk)
        assert np.abs(s - so).max() < SCORE_TOL[dtype], trunk
        assert np.abs(b - bo).max() < SCORE_TOL[dtype], trunk
        # classes outside the active adapters' lists score exactly 0; a frame without adapters is all zero
        assert np.all(s[0, 10:] == 0) and np.all(s[1, :6] == 0) and np.all(s[2] == 0)
    # without base scores no base branch is run (the frame's own slot carries its lowest adapter)
    n0 = m.launch_count()
    s_nb, _ = run_branched(m, w, dtype, L - 2, with_base=False)
    n_nb = m.launch_count() - n0
    assert np.abs(s_nb - so).max() < SCORE_TOL[dtype]
    # frame order does not matter
    perm = [3, 1, 0, 2]
    off_p, ids_p = wl.sets_to_csr([sets[i] for i in perm])
    s_p, b_p = run_branched(m, w, dtype, L - 2, frames=w.frames[perm], offsets=off_p, ids=ids_p)
    assert np.abs(s_p - so[perm]).max() < SCORE_TOL[dtype]
    assert np.abs(b_p - bo[perm]).max() < SCORE_TOL[dtype]
    # the one-stream forward on the same handle is not disturbed by the branch plan
    import torch
    sc = torch.zeros((4, w.spec.n_classes), device="cuda")
    bs = torch.zeros((4, w.spec.n_classes), device="cuda")
    m.forward(frames_to_dev(w.frames, dtype), w.set_offsets, w.set_ids, sc, bs)
    assert m.status() == 0
    assert np.abs(sc.cpu().numpy() - s1).max() < SCORE_TOL[dtype]
    assert np.abs(bs.cpu().numpy() - b1).max() < SCORE_TOL[dtype]
    assert n_nb > 0
    m.close()


def test_branched_deit_small_sampled_rows():
    """64 frames x 1-3 adapters: 64 trunk slots plus one slot per (frame, adapter) branch; several
    128-row tiles per adapter group and a ragged tail."""
    from paper_2507_14959_b200 import binding
    w0 = wl.deit_small_streams()
    spec = w0.spec
    ads = [wl.make_adapter("deit_small_branched", spec, a, 8, np.arange(9 * a, 9 * a + 16),
                           layers=range(spec.layers - 3, spec.layers), ab_std=0.04) for a in range(16)]
    w = wl.Workload("deit_small_branched", spec, w0.backbone, ads, w0.frames, w0.set_offsets, w0.set_ids)
    nnz = int(w.set_offsets[-1])
    m = binding.model_from_workload(w, dtype=0, max_frames=64 + nnz)
    s, b = run_branched(m, w, 0, spec.layers - 3)
    sizes = np.diff(w.set_offsets)
    rows = [0, 63, int(np.argmax(sizes)), int(np.argmin(sizes)), 17, 40]
    so, bo = oracle_branched(w, rows)
    assert np.abs(s[rows] - so).max() < SCORE_TOL[0]
    assert np.abs(b[rows] - bo).max() < SCORE_TOL[0]
    # one slot too few is refused before anything is launched
    m2 = binding.model_from_workload(w, dtype=0, max_frames=64 + nnz - 1)
    n0 = m2.launch_count()
    with pytest.raises(binding.PolymorphError) as e:
        run_branched(m2, w, 0, spec.layers - 3)
    assert e.value.code == binding.PM_ERR_CAPACITY and m2.launch_count() == n0
    m2.close()
    m.close()


def test_branched_argument_errors():
    from paper_2507_14959_b200 import binding
    w = tiny_branch_workload(2, [[0], [1, 3]])
    m = binding.model_from_workload(w, dtype=0, max_frames=8)
    n0 = m.launch_count()
    for trunk, code in [(w.spec.layers - 1, binding.PM_ERR_STATE),      # adapters touch block L-2
                        (-1, binding.PM_ERR_ARG), (w.spec.layers + 1, binding.PM_ERR_ARG)]:
        with pytest.raises(binding.PolymorphError) as e:
            run_branched(m, w, 0, trunk)
        assert e.value.code == code
    off, ids = np.array([0, 2, 3], np.int32), np.array([0, 0, 1], np.int32)      # duplicate id
    with pytest.raises(binding.PolymorphError) as e:
        run_branched(m, w, 0, 10, offsets=off, ids=ids)
    assert e.value.code == binding.PM_ERR_ARG
    assert m.launch_count() == n0
    m.close()
