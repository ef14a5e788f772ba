"""Context construction of the library (Sec. 3.4: co-occurrence counts on the GPU, Algorithm 1 and
Eq. 6 on the host) against the oracle.  Contexts are integer lists: exact equality."""
import numpy as np
import pytest

from oracle import polymorph_oracle as po


def random_label_sets(seed, n_labels, n_frames, max_labels=3, n_themes=6):
    """Frames draw their labels from one of a few themes (overlapping label ranges), like scenes that
    share objects; a few labels never occur."""
    g = np.random.default_rng(seed)
    usable = n_labels - 3
    width = max(4, usable // n_themes + 3)
    sets = []
    for _ in range(n_frames):
        lo = int(g.integers(0, n_themes)) * (usable // n_themes)
        pool = np.arange(lo, min(usable, lo + width))
        k = int(g.integers(1, max_labels + 1))
        sets.append(set(int(x) for x in g.choice(pool, size=min(k, len(pool)), replace=False)))
    return sets


@pytest.mark.parametrize("seed", range(5))
@pytest.mark.parametrize("overlap", [False, True])
def test_build_contexts_and_coherence_match_oracle(seed, overlap):
    from paper_2507_14959_b200 import binding
    K, T = 48, 600
    sets = random_label_sets(seed, K, T)
    co = po.cooccurrence(sets, K)
    g = np.random.default_rng(100 + seed)
    for B, M in [(int(g.integers(2, 8)), int(g.integers(2, 14))), (5, 11), (1, 4), (25, 3)]:
        want = po.build_contexts(co, B, M, overlap)
        got = binding.build_contexts(co, B, M, overlap)
        assert got == want, (B, M)
        assert binding.intra_coherence(got, co / T) == pytest.approx(po.intra_coherence(want, co / T), rel=1e-6)
    assert binding.intra_coherence([], co / T) == 0.0


def test_build_contexts_argument_errors():
    from paper_2507_14959_b200 import binding
    co = np.eye(4, dtype=np.float32)
    for B, M in [(0, 3), (3, 0)]:
        with pytest.raises(binding.PolymorphError) as e:
            binding.build_contexts(co, B, M, False)
        assert e.value.code == binding.PM_ERR_ARG
    with pytest.raises(binding.PolymorphError):
        binding.intra_coherence([[0, 9]], co)           # label out of range


@pytest.mark.gpu
def test_cooccurrence_counts_match_oracle_and_feed_algorithm_1():
    import torch
    from paper_2507_14959_b200 import binding
    K, T = 203, 5000                                    # ragged last label word, many frames
    sets = random_label_sets(7, K, T, max_labels=4, n_themes=11)
    sets[17] = set()                                    # a frame without labels
    sets[18] = set(range(0, 70))                        # more labels than a frame may carry: first 64 counted
    nw = (K + 31) // 32
    bits = np.zeros((T, nw), dtype=np.uint32)
    for f, Y in enumerate(sets):
        for k in Y:
            bits[f, k // 32] |= np.uint32(1) << np.uint32(k % 32)
    lab = torch.from_numpy(bits.view(np.int32)).cuda()
    co = torch.full((K, K), -1.0, device="cuda")
    status = torch.full((1,), 7, dtype=torch.int32, device="cuda")
    binding.cooccurrence(lab, K, co, status)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.PM_ERR_CAPACITY
    sets_counted = list(sets)
    sets_counted[18] = set(range(0, 64))
    want = po.cooccurrence(sets_counted, K)
    np.testing.assert_array_equal(co.cpu().numpy().astype(np.float64), want)
    # second call on the same buffers (overwrites), no oversized frame this time
    sets[18] = {1, 2}
    bits[18] = 0
    bits[18, 0] = 0b110
    lab = torch.from_numpy(bits.view(np.int32)).cuda()
    binding.cooccurrence(lab, K, co, status)
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    want = po.cooccurrence(sets, K)
    got = co.cpu().numpy()
    np.testing.assert_array_equal(got.astype(np.float64), want)
    # the counted matrix drives Algorithm 1 the same way on both sides
    assert binding.build_contexts(got, 8, 40, False) == po.build_contexts(want, 8, 40, False)
    assert binding.build_contexts(got, 8, 40, True) == po.build_contexts(want, 8, 40, True)
