"""Pins for the oracle's Algorithm 2 (context detection): hand-worked cases, exhaustive set
cover on small tables, the coverage constraint (Eq. 2) as a post-condition, Eq. 7 and Eq. 8."""
import itertools

import numpy as np
import pytest

import workloads as wl
from oracle import polymorph_oracle as po


def ones(contexts):
    return [np.ones(len(c), dtype=np.float32) for c in contexts]


def test_threshold_is_strict():
    assert po.labels_from_scores(np.array([0.5, 0.50001, 0.4999, 0.9]), 0.5) == {1, 3}


def test_greedy_prefers_small_contexts_over_cardinality():
    # Y={1,2}: the two singletons are taken before the 3-class context that would cover both.
    contexts = [[1], [2], [1, 2, 3]]
    got = po.detect_contexts({1, 2}, None, contexts, ones(contexts), 0.6, None, False)
    assert got == [0, 1]
    assert po.minimum_cover_size({1, 2}, contexts, ones(contexts), 0.6) == 1


def test_size_order_and_id_tiebreak():
    contexts = [[5, 6, 7], [5, 9], [5, 8]]          # sizes 3, 2, 2 -> order 1, 2, 0
    assert po.context_order(contexts) == [1, 2, 0]
    got = po.detect_contexts({5}, None, contexts, ones(contexts), 0.6, None, False)
    assert got == [1]
    got = po.detect_contexts({5, 7, 8}, None, contexts, ones(contexts), 0.6, None, False)
    assert got == [0, 1, 2]                          # 1 gives 5, 2 gives 8, 0 gives 7


def test_accuracy_threshold_filters_providers():
    contexts = [[1, 2], [1, 2, 3]]
    acc = [np.array([0.9, 0.5]), np.array([0.9, 0.7, 0.7])]
    # label 2 is only provided at >= 0.6 by context 1
    assert po.detect_contexts({2}, None, contexts, acc, 0.6, None, False) == [1]
    assert po.detect_contexts({1, 2}, None, contexts, acc, 0.6, None, False) == [0, 1]
    # tau too high: label undetectable, result empty, no error
    assert po.detect_contexts({2}, None, contexts, acc, 0.95, None, False) == []
    # a_{C,l} == tau counts as provided
    assert po.detect_contexts({2}, None, contexts, acc, 0.5, None, False) == [0]


def test_keep_when_labels_unchanged():
    contexts = [[1], [2], [1, 2, 3]]
    # S_prev is kept as is even though the greedy branch would pick something else
    got = po.detect_contexts({1, 2}, {1, 2}, contexts, ones(contexts), 0.6, [2], False)
    assert got == [2]
    got = po.detect_contexts({1}, {1, 2}, contexts, ones(contexts), 0.6, [2], False)
    assert got == [0]


def test_context_copy_branch():
    contexts = [[1], [2], [1, 2, 3]]
    acc = [np.array([1.0]), np.array([1.0]), np.array([1.0, 0.4, 1.0])]
    # Y changed, copy enabled, S_prev={2} still covers {1,3} at tau -> kept
    assert po.detect_contexts({1, 3}, {1}, contexts, acc, 0.6, [2], True) == [2]
    # label 2 is in context 2 but below tau -> not covered -> greedy
    assert po.detect_contexts({2, 3}, {1}, contexts, acc, 0.6, [2], True) == [1, 2]
    # copy disabled -> greedy
    assert po.detect_contexts({1, 3}, {1}, contexts, acc, 0.6, [2], False) == [0, 2]
    # empty label set: copy keeps the previous set, greedy returns nothing
    assert po.detect_contexts(set(), {1}, contexts, acc, 0.6, [2], True) == [2]
    assert po.detect_contexts(set(), {1}, contexts, acc, 0.6, [2], False) == []


def coverable(Y, contexts, acc, tau):
    return {l for l in Y if any(l in list(c) and acc[i][list(c).index(l)] >= tau
                                for i, c in enumerate(contexts))}


@pytest.mark.parametrize("seed", range(12))
def test_disjoint_tables_greedy_is_the_unique_minimum_cover(seed):
    ctxs, accs = wl.random_cover_table(seed, 8, 16, 4, overlap=False)
    ctxs = [c for c in ctxs if len(c)]
    accs = [a for a in accs if len(a)]
    g = wl.rng_for("Y", seed)
    for _ in range(10):
        Y = set(int(k) for k in g.choice(16, size=int(g.integers(0, 5)), replace=False))
        S = po.detect_contexts(Y, None, ctxs, accs, 0.6, None, False)
        # Eq. 2 post-condition on the coverable labels
        cov = coverable(Y, ctxs, accs, 0.6)
        provided = {int(l) for c in S for j, l in enumerate(ctxs[c]) if accs[c][j] >= 0.6}
        assert cov <= provided
        assert len(S) == po.minimum_cover_size(Y, ctxs, accs, 0.6)
        # unique: exactly the owners of the coverable labels
        owners = {i for i, c in enumerate(ctxs) for l in cov if l in list(c)}
        assert set(S) == owners


@pytest.mark.parametrize("seed", range(12))
def test_overlapping_tables_valid_cover_and_bounds(seed):
    ctxs, accs = wl.random_cover_table(seed, 10, 14, 5, overlap=True)
    g = wl.rng_for("Yo", seed)
    for _ in range(10):
        Y = set(int(k) for k in g.choice(14, size=int(g.integers(0, 5)), replace=False))
        S = po.detect_contexts(Y, None, ctxs, accs, 0.6, None, False)
        cov = coverable(Y, ctxs, accs, 0.6)
        provided = {int(l) for c in S for j, l in enumerate(ctxs[c]) if accs[c][j] >= 0.6}
        assert cov <= provided
        opt = po.minimum_cover_size(Y, ctxs, accs, 0.6)
        assert opt <= len(S) <= len(cov)
        assert S == sorted(set(S))
        # every chosen context is needed at its turn: it is the first provider of some label
        order = po.context_order(ctxs)
        first = {}
        for l in cov:
            for c in order:
                cl = list(ctxs[c])
                if l in cl and accs[c][cl.index(l)] >= 0.6:
                    first[l] = c
                    break
        assert set(S) == set(first.values())


def test_eq7_eq8_hand_example():
    seq = [[0], [0], [0, 2], [2, 0], [1], []]
    assert po.avg_coverage(seq) == pytest.approx(7 / 6)
    assert po.switch_penalty(seq) == 3              # changes at t=3, t=5, t=6
