"""CPU oracle for the Polymorph hot path.  TEST INFRASTRUCTURE ONLY.

This file is the slow, plain statement of what the CUDA library must compute.  It is used by the
tests, by the smoke check and by the benchmark's CPU-baseline leg, and by nothing else: the
product path never imports it.  It shares no code with the CUDA path.

Precision: float64 throughout by default (``dtype=np.float32`` is accepted for timing runs).
The paper does not fix a precision.

What follows the paper and where:
  * lora_linear        Sec. 3.1: h = x(W + AB) = xW + xAB, several adapters summed on top of xW
                       without merging; the adapter scaling (alpha / r, Sec. 4: r = 16, alpha = 32).
  * forward_frame      the cited ViT/DeiT encoder (pre-LN blocks, CLS token, learned positions),
                       every linear of every block being a lora_linear (Fig. 2a).
  * forward_branched   Fig. 2b / Fig. 5b read literally: the base model and each active adapter are
                       separate branches over the frame, merged at the end.
  * heads / compose    Sec. 4 (one head per adapter over its class subset), Fig. 5b (active outputs
                       merged), Sec. 3.2 (base prediction over the full label space).
  * detect_contexts    Algorithm 2, step by step.
  * build_contexts     Algorithm 1 (context construction from label co-occurrence), step by step.
  * intra_coherence    Eq. 6.
  * avg_coverage, switch_penalty   Eq. 7 and Eq. 8.
  * model_stats        the parameter / memory / MAC accounting behind Table 2.

Readings taken where the paper is silent are listed next to each function.

Pins (tests/test_oracle_*.py): merged-weight brute force, a randomly initialised third-party ViT
encoder for the wiring, closed forms for LayerNorm / softmax / GELU, Table 2's printed
differences, exhaustive set cover on small tables.  Behaviour of *trained* models (mAP, F1) is
parity unpinned: no trained weights or datasets exist here.
"""
from __future__ import annotations

import itertools
import math

import numpy as np
from scipy.special import erf as _erf

PROJ = ("qkv", "proj", "fc1", "fc2")


# --------------------------------------------------------------------------------------
# elementary operators (textbook definitions)
# --------------------------------------------------------------------------------------
def layernorm(x, gamma, beta, eps):
    """Row-wise (x - mean) / sqrt(var + eps) * gamma + beta with the biased variance."""
    mu = x.mean(axis=-1, keepdims=True)
    var = ((x - mu) ** 2).mean(axis=-1, keepdims=True)
    return (x - mu) / np.sqrt(var + eps) * gamma + beta


def softmax_rows(s):
    s = s - s.max(axis=-1, keepdims=True)
    e = np.exp(s)
    return e / e.sum(axis=-1, keepdims=True)


def gelu(x):
    """Exact GELU: x * Phi(x)."""
    return 0.5 * x * (1.0 + _erf(x / math.sqrt(2.0)))


def sigmoid(x):
    return 1.0 / (1.0 + np.exp(-x))


# --------------------------------------------------------------------------------------
# Sec. 3.1: the unmerged multi-adapter linear
# --------------------------------------------------------------------------------------
def lora_linear(v, W, b, active):
    """y = v W + b + sum_a s_a (v A_a) B_a.

    ``active`` is a list of (s_a, A_a, B_a) in ascending adapter id; entries whose A is None
    (adapter does not touch this layer/projection) are skipped.  Nothing is merged into W.
    """
    y = v @ W + b
    for s, A, B in active:
        if A is None:
            continue
        y = y + s * ((v @ A) @ B)
    return y


def patchify(frame, patch):
    """[3, H, W] -> [G*G, 3*patch*patch]; patch i = (row i // G, col i % G), vector order
    (channel, y, x)."""
    c, h, w = frame.shape
    g = h // patch
    p = frame.reshape(c, g, patch, g, patch)          # c, gy, py, gx, px
    p = p.transpose(1, 3, 0, 2, 4)                    # gy, gx, c, py, px
    return p.reshape(g * g, c * patch * patch)


def attention(qkv, heads):
    """softmax(q k^T / sqrt(dh)) v per head; qkv columns are ordered [3][heads][dh]."""
    T, d3 = qkv.shape
    d = d3 // 3
    dh = d // heads
    q, k, v = (qkv[:, i * d:(i + 1) * d].reshape(T, heads, dh) for i in range(3))
    out = np.empty((T, heads, dh), dtype=qkv.dtype)
    for h in range(heads):
        s = (q[:, h] @ k[:, h].T) / math.sqrt(dh)
        out[:, h] = softmax_rows(s) @ v[:, h]
    return out.reshape(T, d)


def cls_feature(backbone, frame, adapters_active, heads, patch, ln_eps, dtype=np.float64):
    """Final-LayerNorm CLS feature z of one frame under its active adapters.

    Readings: pre-LN blocks, biases on every linear, CLS at token 0, learned positions added
    after the patch projection, exact-erf GELU, LoRA on qkv/proj/fc1/fc2 of every layer unless an
    adapter leaves a block out (A is None).
    """
    bb = {k: np.asarray(v, dtype=dtype) for k, v in backbone.items()}
    L = bb["qkv_w"].shape[0]
    acts = [(dtype(a.scale),
             [None if m is None else np.asarray(m, dtype=dtype) for m in a.A],
             [None if m is None else np.asarray(m, dtype=dtype) for m in a.B])
            for a in adapters_active]

    def lin(v, l, pi, W, b):
        return lora_linear(v, W, b, [(s, A[l * 4 + pi], B[l * 4 + pi]) for s, A, B in acts])

    p = patchify(np.asarray(frame, dtype=dtype), patch)
    x = np.concatenate([bb["cls"][None, :], p @ bb["patch_w"] + bb["patch_b"]], axis=0) + bb["pos"]
    for l in range(L):
        u = layernorm(x, bb["ln1_g"][l], bb["ln1_b"][l], ln_eps)
        qkv = lin(u, l, 0, bb["qkv_w"][l], bb["qkv_b"][l])
        x = x + lin(attention(qkv, heads), l, 1, bb["proj_w"][l], bb["proj_b"][l])
        u = layernorm(x, bb["ln2_g"][l], bb["ln2_b"][l], ln_eps)
        hmid = gelu(lin(u, l, 2, bb["fc1_w"][l], bb["fc1_b"][l]))
        x = x + lin(hmid, l, 3, bb["fc2_w"][l], bb["fc2_b"][l])
    return layernorm(x[0], bb["lnf_g"], bb["lnf_b"], ln_eps)


def compose_scores(z, adapters_active, n_classes):
    """Per-adapter heads, sigmoid, merge (Fig. 5b, Sec. 4).

    Reading: each active adapter scores only its own class subset; a class listed by several
    active adapters takes the maximum; a class listed by no active adapter scores 0 (the label
    space of a frame is restricted to its active contexts, Sec. 4 discussion of Fig. 8).
    """
    scores = np.zeros(n_classes, dtype=z.dtype)
    for a in adapters_active:
        p = sigmoid(z @ np.asarray(a.head_w, dtype=z.dtype) + np.asarray(a.head_b, dtype=z.dtype))
        for j, k in enumerate(a.class_ids):
            scores[k] = max(scores[k], p[j])
    return scores


def forward(backbone, adapters, frames, set_offsets, set_ids, heads, patch, ln_eps, n_classes,
            dtype=np.float64):
    """scores[F, K] (composed adapter heads) and base_scores[F, K] (base head on the same z)."""
    F = len(set_offsets) - 1
    scores = np.zeros((F, n_classes), dtype=dtype)
    base = np.zeros((F, n_classes), dtype=dtype)
    for f in range(F):
        ids = sorted(int(i) for i in set_ids[set_offsets[f]:set_offsets[f + 1]])
        act = [adapters[i] for i in ids]
        z = cls_feature(backbone, frames[f], act, heads, patch, ln_eps, dtype)
        base[f] = sigmoid(z @ np.asarray(backbone["head_w"], dtype=dtype)
                          + np.asarray(backbone["head_b"], dtype=dtype))
        scores[f] = compose_scores(z, act, n_classes)
    return scores, base


def forward_branched(backbone, adapters, frames, set_offsets, set_ids, heads, patch, ln_eps, n_classes,
                     dtype=np.float64):
    """The per-adapter-branch reading of Fig. 2b / Fig. 5b: the base model and every active adapter
    process the frame as separate models (each adapter alone on top of the shared backbone), every
    adapter's head reads its own branch, and the branch outputs are merged as in compose_scores.

    base_scores[f] comes from the branch without any adapter (the plain base model of Sec. 3.2);
    scores[f, k] = max over active adapters a listing k of adapter a's own score, 0 otherwise.
    Nothing is shared between branches here: each one is a complete forward of its own, so the
    result does not depend on where an implementation lets the branches split.
    """
    F = len(set_offsets) - 1
    scores = np.zeros((F, n_classes), dtype=dtype)
    base = np.zeros((F, n_classes), dtype=dtype)
    for f in range(F):
        z0 = cls_feature(backbone, frames[f], [], heads, patch, ln_eps, dtype)
        base[f] = sigmoid(z0 @ np.asarray(backbone["head_w"], dtype=dtype)
                          + np.asarray(backbone["head_b"], dtype=dtype))
        for i in sorted(int(i) for i in set_ids[set_offsets[f]:set_offsets[f + 1]]):
            za = cls_feature(backbone, frames[f], [adapters[i]], heads, patch, ln_eps, dtype)
            scores[f] = np.maximum(scores[f], compose_scores(za, [adapters[i]], n_classes))
    return scores, base


# --------------------------------------------------------------------------------------
# Algorithm 2: greedy context detection with conditional context copy
# --------------------------------------------------------------------------------------
def labels_from_scores(scores_row, thr):
    """Y_t = {k : score_k > thr} (strict)."""
    return {int(k) for k in np.nonzero(np.asarray(scores_row) > thr)[0]}


def context_order(contexts):
    """Contexts in order of increasing size |C| (all listed classes); ties by ascending id."""
    return sorted(range(len(contexts)), key=lambda c: (len(contexts[c]), c))


def detect_contexts(Y_t, Y_prev, contexts, acc, tau, S_prev, context_copy):
    """Algorithm 2.  ``contexts[c]`` is the class-id list of context c, ``acc[c][j]`` the
    accuracy a_{C,l} of its j-th class.  Y_prev / S_prev are None on the first frame of a stream
    (then the greedy branch runs).  Returns the sorted list of selected context ids.

    Labels that no context provides at accuracy >= tau stay uncovered (Sec. 3.5, last paragraph).
    """
    Y_t = set(Y_t)

    def provides(c, l):
        cl = list(contexts[c])
        return l in cl and acc[c][cl.index(l)] >= tau

    if Y_prev is not None and S_prev is not None and Y_t == set(Y_prev):
        return sorted(S_prev)
    if (context_copy and S_prev is not None
            and all(any(provides(c, l) for c in S_prev) for l in Y_t)):
        return sorted(S_prev)
    S, U = [], set(Y_t)
    if not U:
        return S
    for c in context_order(contexts):
        prov = {l for l in U if provides(c, l)}
        if prov:
            S.append(c)
            U -= prov
            if not U:
                break
    return sorted(S)


def minimum_cover_size(Y, contexts, acc, tau):
    """Exhaustive search: the smallest number of contexts covering every coverable label of Y
    at accuracy >= tau (checker for small tables)."""
    def prov(c):
        return {int(l) for j, l in enumerate(contexts[c]) if acc[c][j] >= tau} & set(Y)
    provs = [prov(c) for c in range(len(contexts))]
    target = set().union(*provs) if provs else set()
    if not target:
        return 0
    for n in range(1, len(contexts) + 1):
        for comb in itertools.combinations(range(len(contexts)), n):
            if set().union(*(provs[c] for c in comb)) >= target:
                return n
    raise AssertionError("unreachable")


# --------------------------------------------------------------------------------------
# Algorithm 1: context construction from a label co-occurrence matrix, and Eq. 6
# --------------------------------------------------------------------------------------
def cooccurrence(label_sets, n_labels):
    """co[i, j] = number of frames whose label set holds both i and j (diagonal: frames holding i).
    Sec. 3.4: the matrix is built from the training set's per-frame label sets."""
    co = np.zeros((n_labels, n_labels), dtype=np.float64)
    for Y in label_sets:
        for i in Y:
            for j in Y:
                co[i, j] += 1.0
    return co


def build_contexts(co, B, M_max, allow_overlap):
    """Algorithm 1 (BuildContexts), step by step.  Returns the contexts as sorted label lists, in the
    order they were created.

    Readings where the listing is silent:
      * valid labels = labels that occur at all (co[l, l] > 0);
      * they are visited from the most to the least frequent (Sec. 3.4: clusters are centred on
        frequently occurring labels), ties by ascending label;
      * the cluster around l = l plus its up to B-1 strongest co-occurring valid neighbours with
        co[l, j] > 0 (ties by ascending label); without overlap, labels already assigned are no
        candidates;
      * unique = not equal, as a set, to a context already kept;
      * an uncovered label (visited in ascending order) goes to the context with room left whose
        members co-occur with it most in total, ties by the earlier context; if no context has
        room it stays uncovered (the size limit wins).
    """
    co = np.asarray(co, dtype=np.float64)
    K = co.shape[0]
    valid = [l for l in range(K) if co[l, l] > 0]
    order = sorted(valid, key=lambda l: (-co[l, l], l))
    contexts, assigned = [], set()
    for l in order:
        if not allow_overlap and l in assigned:
            continue
        cand = [j for j in valid if j != l and co[l, j] > 0 and (allow_overlap or j not in assigned)]
        cand.sort(key=lambda j: (-co[l, j], j))
        cluster = sorted([l] + cand[:max(B - 1, 0)])
        if cluster not in contexts and len(contexts) < M_max:
            contexts.append(cluster)
            if not allow_overlap:
                assigned |= set(cluster)
    covered = set().union(*contexts) if contexts else set()
    for l in valid:
        if l in covered:
            continue
        best, best_fit = -1, -1.0
        for c, ctx in enumerate(contexts):
            if len(ctx) >= B:
                continue
            fit = sum(co[l, j] for j in ctx)
            if fit > best_fit:
                best, best_fit = c, fit
        if best >= 0:
            contexts[best] = sorted(contexts[best] + [l])
            covered.add(l)
    return contexts


def intra_coherence(contexts, co_norm):
    """Eq. 6: mean over contexts of the mean normalised co-occurrence over ordered pairs i != j of the
    context.  Reading: a context with a single label has no pair and contributes 0."""
    if not contexts:
        return 0.0
    total = 0.0
    for ctx in contexts:
        n = len(ctx)
        if n < 2:
            continue
        s = 0.0
        for i in ctx:
            for j in ctx:
                if i != j:
                    s += co_norm[i][j]
        total += s / (n * (n - 1))
    return total / len(contexts)


def avg_coverage(S_seq):
    """Eq. 7: mean number of active contexts per frame."""
    return sum(len(s) for s in S_seq) / len(S_seq)


def switch_penalty(S_seq):
    """Eq. 8: number of t >= 2 with S_t != S_{t-1}."""
    return sum(1 for t in range(1, len(S_seq)) if sorted(S_seq[t]) != sorted(S_seq[t - 1]))


# --------------------------------------------------------------------------------------
# Table 2 accounting
# --------------------------------------------------------------------------------------
def model_stats(d, layers, mlp, tokens, patch_dim, n_classes,
                n_adapters=0, rank=0, lora_layers=0, lora_projs_per_layer=0,
                classes_per_adapter=0, active_adapters=0):
    """Parameters, fp32 MiB and multiply-accumulates per frame.

    Base: patch projection, CLS, positions, `layers` blocks (2 LayerNorms, qkv, proj, fc1, fc2
    with biases), final LayerNorm, K-way head.  MACs count the linear maps only.  Each adapter
    adds 2*d*rank parameters per adapted d->d projection plus a (d+1)*classes head; each active
    adapter adds tokens*2*d*rank MACs per adapted projection.
    """
    per_layer = 2 * 2 * d + (d * 3 * d + 3 * d) + (d * d + d) + (d * mlp + mlp) + (mlp * d + d)
    base_params = (patch_dim * d + d) + d + tokens * d + layers * per_layer + 2 * d \
        + d * n_classes + n_classes
    base_macs = (tokens - 1) * patch_dim * d + tokens * layers * (4 * d * d + 2 * d * mlp) \
        + d * n_classes
    lora_params_each = lora_layers * lora_projs_per_layer * 2 * d * rank \
        + (d * classes_per_adapter + classes_per_adapter)
    lora_macs_each = tokens * lora_layers * lora_projs_per_layer * 2 * d * rank
    params = base_params + n_adapters * lora_params_each
    macs = base_macs + active_adapters * lora_macs_each
    return {"params": params, "mib_fp32": params * 4 / 2 ** 20, "macs": macs}
