"""Pins for the forward part of the CPU oracle: each test checks it against something the paper
or the mathematics fixes, never against the oracle itself."""
import math
import os

import numpy as np
import pytest

import workloads as wl
from oracle import polymorph_oracle as po

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def small_spec(layers=2, n_classes=12):
    return wl.ModelSpec(img=48, d=32, heads=2, mlp=64, n_classes=n_classes, layers=layers)


def small_model(name="pin_small", layers=2, ranks=(4, 8, 2)):
    spec = small_spec(layers)
    bb = wl.make_backbone(name, spec)
    ads = [wl.make_adapter(name, spec, a, r, np.arange(4 * a, 4 * a + 4), ab_std=0.2)
           for a, r in enumerate(ranks)]
    return spec, bb, ads


# ---------------------------------------------------------------- elementary operators
def test_layernorm_closed_forms():
    g = np.linspace(0.5, 1.5, 8)
    b = np.linspace(-1, 1, 8)
    const = np.full((3, 8), 4.25)
    np.testing.assert_allclose(po.layernorm(const, g, b, 1e-6), np.tile(b, (3, 1)), atol=1e-12)
    # two-valued row: mean 0, biased variance 1 -> output = +-gamma/sqrt(1+eps) + beta
    row = np.array([[1.0, -1.0] * 4])
    want = row / math.sqrt(1 + 1e-6) * g + b
    np.testing.assert_allclose(po.layernorm(row, g, b, 1e-6), want, atol=1e-12)


def test_layernorm_against_torch():
    import torch
    x = wl.rng_for("ln").standard_normal((5, 24))
    g = wl.rng_for("ln_g").standard_normal(24)
    b = wl.rng_for("ln_b").standard_normal(24)
    ref = torch.nn.functional.layer_norm(torch.from_numpy(x), (24,), torch.from_numpy(g),
                                         torch.from_numpy(b), 1e-6).numpy()
    np.testing.assert_allclose(po.layernorm(x, g, b, 1e-6), ref, atol=1e-12)


def test_gelu_closed_forms():
    phi1 = 0.8413447460685429      # standard normal CDF at 1
    assert po.gelu(np.array(0.0)) == 0.0
    assert abs(po.gelu(np.array(1.0)) - phi1) < 1e-15
    assert abs(po.gelu(np.array(-1.0)) + (1 - phi1)) < 1e-15
    assert abs(po.gelu(np.array(10.0)) - 10.0) < 1e-12
    assert abs(po.gelu(np.array(-10.0))) < 1e-12


def test_attention_special_cases():
    T, H, dh = 7, 2, 4
    d = H * dh
    g = wl.rng_for("attn")
    qkv = g.standard_normal((T, 3 * d))
    # identical keys -> uniform softmax -> every query returns the mean of V
    qkv_same = qkv.copy()
    qkv_same[:, d:2 * d] = qkv[0, d:2 * d]
    out = po.attention(qkv_same, H)
    np.testing.assert_allclose(out, np.tile(qkv[:, 2 * d:].mean(0), (T, 1)), atol=1e-12)
    # against torch's scaled-dot-product attention
    import torch
    t = torch.from_numpy(qkv).reshape(T, 3, H, dh).permute(1, 2, 0, 3)
    ref = torch.nn.functional.scaled_dot_product_attention(t[0], t[1], t[2])
    ref = ref.permute(1, 0, 2).reshape(T, d).numpy()
    np.testing.assert_allclose(po.attention(qkv, H), ref, atol=1e-12)


def test_patchify_matches_strided_convolution():
    import torch
    g = wl.rng_for("patchify")
    frame = g.standard_normal((3, 48, 48))
    w = g.standard_normal((5, 3, 16, 16))
    ref = torch.nn.functional.conv2d(torch.from_numpy(frame)[None], torch.from_numpy(w), stride=16)
    ref = ref[0].flatten(1).T.numpy()                      # [patches, 5], row-major over (gy, gx)
    got = po.patchify(frame, 16) @ w.reshape(5, -1).T
    np.testing.assert_allclose(got, ref, atol=1e-10)


# ---------------------------------------------------------------- wiring vs an independent ViT
def test_plain_backbone_matches_third_party_vit():
    """Empty adapter set == plain backbone: compared with a randomly initialised Hugging Face
    ViT encoder (independent code) carrying the same weights."""
    torch = pytest.importorskip("torch")
    tr = pytest.importorskip("transformers")
    spec = small_spec(layers=3)
    bb = wl.make_backbone("hf_pin", spec)
    cfg = tr.ViTConfig(hidden_size=spec.d, num_hidden_layers=spec.layers,
                       num_attention_heads=spec.heads, intermediate_size=spec.mlp,
                       image_size=spec.img, patch_size=spec.patch, layer_norm_eps=spec.ln_eps,
                       hidden_act="gelu", qkv_bias=True, hidden_dropout_prob=0.0,
                       attention_probs_dropout_prob=0.0)
    m = tr.ViTModel(cfg, add_pooling_layer=False).double().eval()
    sd = {}
    T = lambda a: torch.from_numpy(np.asarray(a, dtype=np.float64))
    d = spec.d
    sd["embeddings.cls_token"] = T(bb["cls"]).reshape(1, 1, d)
    sd["embeddings.position_embeddings"] = T(bb["pos"]).reshape(1, spec.tokens, d)
    sd["embeddings.patch_embeddings.projection.weight"] = T(bb["patch_w"].T).reshape(d, 3, 16, 16)
    sd["embeddings.patch_embeddings.projection.bias"] = T(bb["patch_b"])
    for l in range(spec.layers):
        p = f"encoder.layer.{l}."
        for i, n in enumerate(("query", "key", "value")):
            sd[p + f"attention.attention.{n}.weight"] = T(bb["qkv_w"][l][:, i * d:(i + 1) * d].T)
            sd[p + f"attention.attention.{n}.bias"] = T(bb["qkv_b"][l][i * d:(i + 1) * d])
        sd[p + "attention.output.dense.weight"] = T(bb["proj_w"][l].T)
        sd[p + "attention.output.dense.bias"] = T(bb["proj_b"][l])
        sd[p + "intermediate.dense.weight"] = T(bb["fc1_w"][l].T)
        sd[p + "intermediate.dense.bias"] = T(bb["fc1_b"][l])
        sd[p + "output.dense.weight"] = T(bb["fc2_w"][l].T)
        sd[p + "output.dense.bias"] = T(bb["fc2_b"][l])
        sd[p + "layernorm_before.weight"] = T(bb["ln1_g"][l])
        sd[p + "layernorm_before.bias"] = T(bb["ln1_b"][l])
        sd[p + "layernorm_after.weight"] = T(bb["ln2_g"][l])
        sd[p + "layernorm_after.bias"] = T(bb["ln2_b"][l])
    sd["layernorm.weight"] = T(bb["lnf_g"])
    sd["layernorm.bias"] = T(bb["lnf_b"])
    missing, unexpected = m.load_state_dict(sd, strict=False)
    assert not unexpected and not missing, (missing, unexpected)
    frames = wl.make_frames("hf_pin", spec, 2)
    with torch.no_grad():
        ref = m(pixel_values=torch.from_numpy(frames).double()).last_hidden_state[:, 0].numpy()
    for f in range(2):
        z = po.cls_feature(bb, frames[f], [], spec.heads, spec.patch, spec.ln_eps)
        np.testing.assert_allclose(z, ref[f], atol=1e-9)
    # the scores of a frame with no active adapter: base head on that feature, composed row zero
    off, ids = wl.sets_to_csr([[], []])
    scores, base = po.forward(bb, [], frames, off, ids, spec.heads, spec.patch, spec.ln_eps,
                              spec.n_classes)
    want = 1 / (1 + np.exp(-(ref @ bb["head_w"].astype(np.float64) + bb["head_b"])))
    np.testing.assert_allclose(base, want, atol=1e-9)
    assert np.all(scores == 0)


# ---------------------------------------------------------------- Sec. 3.1 identity
def merged_backbone(spec, bb, ads):
    """Brute force W' = W + sum_a s_a A_a B_a for every adapted (layer, projection)."""
    out = {k: np.asarray(v, dtype=np.float64).copy() for k, v in bb.items()}
    for a in ads:
        for l in range(spec.layers):
            for pi, p in enumerate(wl.PROJ_NAMES):
                if a.A[l * 4 + pi] is None:
                    continue
                A = a.A[l * 4 + pi].astype(np.float64)
                B = a.B[l * 4 + pi].astype(np.float64)
                W = out[p + "_w"][l]
                for i in range(W.shape[0]):          # explicit loops: no shared matmul shortcut
                    W[i] += a.scale * (A[i][:, None] * B).sum(0)
    return out


@pytest.mark.parametrize("active", [[0], [1, 2], [0, 1, 2]])
def test_unmerged_equals_merged_weights(active):
    spec, bb, ads = small_model()
    frame = wl.make_frames("pin_small", spec, 1)[0]
    act = [ads[i] for i in active]
    z_unmerged = po.cls_feature(bb, frame, act, spec.heads, spec.patch, spec.ln_eps)
    z_merged = po.cls_feature(merged_backbone(spec, bb, act), frame, [], spec.heads, spec.patch,
                              spec.ln_eps)
    z_plain = po.cls_feature(bb, frame, [], spec.heads, spec.patch, spec.ln_eps)
    np.testing.assert_allclose(z_unmerged, z_merged, atol=1e-10)
    assert np.abs(z_unmerged - z_plain).max() > 1e-2      # the adapters do change the result


def test_partial_adapter_matches_merged_and_zero_B_is_identity():
    spec = small_spec()
    name = "pin_partial"
    bb = wl.make_backbone(name, spec)
    # query/value-style special case: only the qkv projection of the last layer is adapted
    a = wl.make_adapter(name, spec, 0, 4, np.arange(4), layers=[spec.layers - 1], projs=("qkv",),
                        ab_std=0.2)
    frame = wl.make_frames(name, spec, 1)[0]
    z1 = po.cls_feature(bb, frame, [a], spec.heads, spec.patch, spec.ln_eps)
    z2 = po.cls_feature(merged_backbone(spec, bb, [a]), frame, [], spec.heads, spec.patch, spec.ln_eps)
    np.testing.assert_allclose(z1, z2, atol=1e-10)
    for i, m in enumerate(a.B):
        if m is not None:
            a.B[i] = np.zeros_like(m)
    z0 = po.cls_feature(bb, frame, [a], spec.heads, spec.patch, spec.ln_eps)
    zp = po.cls_feature(bb, frame, [], spec.heads, spec.patch, spec.ln_eps)
    np.testing.assert_allclose(z0, zp, atol=1e-13)


def test_lora_linear_scale_is_alpha_over_rank():
    """Sec. 4: rank 16 with scaling factor 32 -> every adapter term is multiplied by 2."""
    spec = small_spec()
    a = wl.make_adapter("scale_pin", spec, 0, 16, np.arange(4))
    assert a.scale == 2.0
    g = wl.rng_for("scale_pin_x")
    v = g.standard_normal((3, spec.d))
    W = g.standard_normal((spec.d, 3 * spec.d))
    b = g.standard_normal(3 * spec.d)
    y = po.lora_linear(v, W, b, [(a.scale, a.A[0].astype(np.float64), a.B[0].astype(np.float64))])
    want = v @ (W + 2.0 * a.A[0].astype(np.float64) @ a.B[0].astype(np.float64)) + b
    np.testing.assert_allclose(y, want, atol=1e-12)


# ---------------------------------------------------------------- batch-level invariants
def test_forward_frame_permutation_and_duplicates():
    spec, bb, ads = small_model()
    frames = wl.make_frames("pin_small", spec, 3)
    frames = np.concatenate([frames, frames[:1]], axis=0)        # frame 3 duplicates frame 0
    sets = [[0], [1, 2], [], [0]]
    off, ids = wl.sets_to_csr(sets)
    s, b = po.forward(bb, ads, frames, off, ids, spec.heads, spec.patch, spec.ln_eps, spec.n_classes)
    np.testing.assert_array_equal(s[0], s[3])
    perm = [2, 0, 3, 1]
    off2, ids2 = wl.sets_to_csr([sets[i] for i in perm])
    s2, b2 = po.forward(bb, ads, frames[perm], off2, ids2, spec.heads, spec.patch, spec.ln_eps,
                        spec.n_classes)
    np.testing.assert_array_equal(s2, s[perm])
    np.testing.assert_array_equal(b2, b[perm])
    # unordered ids in the CSR give the same result as sorted ids
    s3, _ = po.forward(bb, ads, frames[1:2], np.array([0, 2], np.int32), np.array([2, 1], np.int32),
                       spec.heads, spec.patch, spec.ln_eps, spec.n_classes)
    np.testing.assert_array_equal(s3[0], s[1])


def test_compose_hand_case():
    class Ad:
        pass
    z = np.array([1.0, -2.0])
    a0, a1 = Ad(), Ad()
    a0.class_ids = np.array([0, 3]); a0.head_w = np.array([[1.0, 0.0], [0.0, 1.0]]); a0.head_b = np.array([0.0, 0.0])
    a1.class_ids = np.array([3, 4]); a1.head_w = np.array([[2.0, 0.0], [0.0, 0.0]]); a1.head_b = np.array([0.0, 1.0])
    sg = lambda t: 1 / (1 + math.exp(-t))
    s = po.compose_scores(z, [a0, a1], 6)
    # class 0: a0 only; class 3: max(a0: sigma(-2), a1: sigma(2)); class 4: a1; others uncovered
    np.testing.assert_allclose(s, [sg(1.0), 0, 0, sg(2.0), sg(1.0), 0], atol=1e-15)
    np.testing.assert_allclose(po.compose_scores(z, [a1, a0], 6), s, atol=0)


def test_branched_forward_equals_distinct_merged_models():
    """Sec. 3.1: merging the adapters means instantiating one distinct model per adapter.  The
    branch reading (Fig. 2b, Fig. 5b) must therefore equal: the plain base model for the base
    scores, and for every active adapter a plain model with W + s A B (brute force) whose feature
    feeds that adapter's own head; maximum where two active adapters list a class."""
    spec = small_spec(n_classes=10)
    name = "pin_branch"
    bb = wl.make_backbone(name, spec)
    # overlapping class lists so that the merge matters: {0..4}, {3..7}, {6..9}
    ads = [wl.make_adapter(name, spec, a, r, np.arange(lo, hi), ab_std=0.2)
           for a, (r, lo, hi) in enumerate([(4, 0, 5), (8, 3, 8), (2, 6, 10)])]
    frames = wl.make_frames(name, spec, 3)
    sets = [[0, 1], [], [2, 0, 1]]
    off, ids = wl.sets_to_csr(sets)
    s, b = po.forward_branched(bb, ads, frames, off, ids, spec.heads, spec.patch, spec.ln_eps,
                               spec.n_classes)
    sg = lambda t: 1.0 / (1.0 + math.exp(-t))
    for f, st in enumerate(sets):
        z0 = po.cls_feature(bb, frames[f], [], spec.heads, spec.patch, spec.ln_eps)
        want_b = [sg(float(z0 @ bb["head_w"][:, k].astype(np.float64) + bb["head_b"][k]))
                  for k in range(spec.n_classes)]
        np.testing.assert_allclose(b[f], want_b, atol=1e-12)
        want = np.zeros(spec.n_classes)
        for a in st:
            za = po.cls_feature(merged_backbone(spec, bb, [ads[a]]), frames[f], [], spec.heads,
                                spec.patch, spec.ln_eps)
            for j, k in enumerate(ads[a].class_ids):
                v = sg(float(za @ ads[a].head_w[:, j].astype(np.float64) + ads[a].head_b[j]))
                want[k] = max(want[k], v)
        np.testing.assert_allclose(s[f], want, atol=1e-10)
    # it is a different function from the one-stream forward whenever two adapters are active ...
    s1, b1 = po.forward(bb, ads, frames, off, ids, spec.heads, spec.patch, spec.ln_eps, spec.n_classes)
    assert np.abs(s1[0] - s[0]).max() > 1e-4 and np.abs(b1[0] - b[0]).max() > 1e-4
    # ... and the same function for a frame without adapters
    np.testing.assert_array_equal(s1[1], s[1])
    np.testing.assert_array_equal(b1[1], b[1])


def test_branched_forward_single_adapter_equals_one_stream_scores():
    spec, bb, ads = small_model()
    frames = wl.make_frames("pin_small", spec, 2)
    off, ids = wl.sets_to_csr([[1], [2]])
    s, b = po.forward_branched(bb, ads, frames, off, ids, spec.heads, spec.patch, spec.ln_eps, spec.n_classes)
    s1, _ = po.forward(bb, ads, frames, off, ids, spec.heads, spec.patch, spec.ln_eps, spec.n_classes)
    off0, ids0 = wl.sets_to_csr([[], []])
    _, b0 = po.forward(bb, ads, frames, off0, ids0, spec.heads, spec.patch, spec.ln_eps, spec.n_classes)
    np.testing.assert_allclose(s, s1, atol=1e-13)
    np.testing.assert_allclose(b, b0, atol=1e-13)


# ---------------------------------------------------------------- Table 2
def read_table2():
    rows = {}
    with open(os.path.join(GOLDEN, "table2.txt")) as fh:
        for line in fh:
            if line.startswith("#") or not line.strip():
                continue
            name, p, m, c = line.split()
            rows[name] = (float(p), float(m), float(c))
    return rows


def test_table2_differences():
    """Table 2: Polymorph minus Base = the 11 adapters (rank 16 on query+value of the last 2 of
    12 layers, 5-class heads) in parameters and fp32 MiB, and ONE active adapter in MACs."""
    t = read_table2()
    kw = dict(d=192, layers=12, mlp=768, tokens=197, patch_dim=768, n_classes=80)
    base = po.model_stats(**kw)
    poly = po.model_stats(**kw, n_adapters=11, rank=16, lora_layers=2, lora_projs_per_layer=2,
                          classes_per_adapter=5, active_adapters=1)
    assert round(base["params"] / 1e6, 2) == t["Base"][0]
    assert round(poly["params"] / 1e6, 2) == t["Polymorph"][0]
    assert abs((poly["params"] - base["params"]) / 1e6 - (t["Polymorph"][0] - t["Base"][0])) < 0.005
    assert abs((poly["mib_fp32"] - base["mib_fp32"]) - (t["Polymorph"][1] - t["Base"][1])) < 0.005
    assert abs((poly["macs"] - base["macs"]) / 1e6 - (t["Polymorph"][2] - t["Base"][2])) < 0.005
    assert abs(base["mib_fp32"] - t["Base"][1]) < 0.02
    # absolute MACs: the table's counter includes a few non-linear-map operations; within 0.5 %
    assert abs(base["macs"] / 1e6 - t["Base"][2]) / t["Base"][2] < 0.005
    larger = po.model_stats(d=768, layers=12, mlp=3072, tokens=197, patch_dim=768, n_classes=80)
    assert round(larger["params"] / 1e6, 2) == t["Larger"][0]
    assert abs(larger["macs"] / 1e6 - t["Larger"][2]) / t["Larger"][2] < 0.005
