"""Pins for the oracle's Algorithm 1 (context construction) and Eq. 6: hand-worked cases, the
constraints the paper states (Sec. 3.3 / 3.4: every valid label covered when there is room, no
context larger than B, at most M_max contexts, unique clusters, disjoint contexts without overlap),
and a co-occurrence structure whose right answer is known by construction."""
import itertools

import numpy as np
import pytest

from oracle import polymorph_oracle as po


def block_cooccurrence(groups, n_labels, within=10.0, across=0.0, freq=None):
    co = np.full((n_labels, n_labels), across)
    for g in groups:
        for i in g:
            for j in g:
                co[i, j] = within
    for l in range(n_labels):
        co[l, l] = (freq[l] if freq is not None else 20.0)
    return co


def test_cooccurrence_counts_hand_case():
    co = po.cooccurrence([{0, 1}, {1}, {0, 1, 3}], 4)
    want = np.array([[2, 2, 0, 1], [2, 3, 0, 1], [0, 0, 0, 0], [1, 1, 0, 1]], dtype=float)
    np.testing.assert_array_equal(co, want)


def test_build_contexts_hand_case_without_overlap():
    # labels 0..5; label 5 never occurs (not valid).  Frequencies: 0 > 3 > 1 > 2 > 4.
    co = np.array([[9, 5, 1, 0, 0, 0],
                   [5, 6, 4, 0, 0, 0],
                   [1, 4, 5, 2, 0, 0],
                   [0, 0, 2, 8, 3, 0],
                   [0, 0, 0, 3, 4, 0],
                   [0, 0, 0, 0, 0, 0]], dtype=float)
    # B = 2: around 0 -> {0, 1} (strongest neighbour 1); around 3 -> {3, 4} (2 is free too but weaker: 2 < 3);
    # 1 assigned; around 2 -> neighbours 1, 3 assigned, 0 assigned -> {2}; 4 assigned.
    assert po.build_contexts(co, 2, 10, False) == [[0, 1], [3, 4], [2]]
    # M_max = 2: {2} cannot be added; 2 is uncovered and no context has room -> stays uncovered
    assert po.build_contexts(co, 2, 2, False) == [[0, 1], [3, 4]]
    # B = 3, M_max = 1: {0, 1, 2} is full; 3 and 4 stay uncovered
    assert po.build_contexts(co, 3, 1, False) == [[0, 1, 2]]
    # B = 4, M_max = 1: {0, 1, 2} has room: 3 fits (co with 2), then the context is full and 4 stays out
    assert po.build_contexts(co, 4, 1, False) == [[0, 1, 2, 3]]


def test_build_contexts_hand_case_with_overlap():
    co = np.array([[9, 5, 1, 0],
                   [5, 6, 4, 0],
                   [1, 4, 5, 2],
                   [0, 0, 2, 8]], dtype=float)
    # order by frequency: 0 (9), 3 (8), 1 (6), 2 (5).  B = 2:
    # 0 -> {0,1}; 3 -> {2,3}; 1 -> {0,1} again: not unique, dropped; 2 -> {1,2}
    assert po.build_contexts(co, 2, 10, True) == [[0, 1], [2, 3], [1, 2]]


def test_build_contexts_recovers_planted_groups():
    groups = [[0, 1, 2, 3], [4, 5, 6], [7, 8, 9, 10, 11]]
    co = block_cooccurrence(groups, 12)
    got = po.build_contexts(co, 5, 10, False)
    assert sorted(got) == sorted(groups)
    # with overlap allowed every label of a group rebuilds the same cluster: still unique
    assert sorted(po.build_contexts(co, 5, 10, True)) == sorted(groups)
    # Eq. 6 on the planted structure: all pairs inside a context co-occur with weight 10 / 20
    assert po.intra_coherence(got, co / 20.0) == pytest.approx(0.5)


@pytest.mark.parametrize("seed", range(6))
@pytest.mark.parametrize("overlap", [False, True])
def test_build_contexts_constraints_on_random_matrices(seed, overlap):
    g = np.random.default_rng(seed)
    K, T = 30, 200
    sets = [set(g.choice(K - 3, size=int(g.integers(1, 4)), replace=False).tolist()) for _ in range(T)]
    co = po.cooccurrence(sets, K)                     # labels K-3 .. K-1 never occur
    B, M = int(g.integers(2, 7)), int(g.integers(3, 12))
    ctxs = po.build_contexts(co, B, M, overlap)
    valid = {l for l in range(K) if co[l, l] > 0}
    assert 0 < len(ctxs) <= M
    assert all(1 <= len(c) <= B and c == sorted(set(c)) and set(c) <= valid for c in ctxs)
    assert len({tuple(c) for c in ctxs}) == len(ctxs)                       # unique
    if not overlap:
        assert sum(len(c) for c in ctxs) == len(set().union(*ctxs))         # disjoint
    uncovered = valid - set().union(*ctxs)
    if uncovered:                                     # only possible when every context is full
        assert all(len(c) == B for c in ctxs)


def test_intra_coherence_hand_case():
    co = np.array([[0, .2, .4], [.2, 0, .6], [.4, .6, 0]])
    # context {0,1,2}: mean over 6 ordered pairs = 0.4; context {0,1}: 0.2; singleton: 0
    assert po.intra_coherence([[0, 1, 2], [0, 1], [2]], co) == pytest.approx((0.4 + 0.2 + 0.0) / 3)
    brute = np.mean([np.mean([co[i][j] for i, j in itertools.permutations(c, 2)]) for c in ([0, 1, 2], [1, 2])])
    assert po.intra_coherence([[0, 1, 2], [1, 2]], co) == pytest.approx(brute)
