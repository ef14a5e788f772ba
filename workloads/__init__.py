"""Seeded synthetic inputs for the Polymorph hot path.

This module only *draws* inputs (frames, weights, adapters, class subsets, accuracy tables,
per-frame adapter sets).  It contains none of the method's arithmetic, so that both the CPU
oracle and the CUDA library can be fed the very same arrays without sharing any code.

Every tensor gets its own sub-seed derived from (master seed, workload name, tensor name), so
generation order never matters.  All floating-point model inputs are rounded once to bf16
(round-to-nearest-even) and handed out as float32 holding exactly representable values; the GPU
stores them as bf16 without further rounding and the oracle widens them to its own precision.

The workloads stand in for the paper's COCO-trained weights and TAO video clips (Sec. 4), which
are not available: at most ~3 labels per frame (Sec. 1), contexts of 5-25 labels (Table 3),
several hundred classes (Sec. 4), slowly changing adapter sets (temporal continuity, Sec. 1).
"""
from __future__ import annotations

import hashlib
from dataclasses import dataclass, field

import numpy as np

MASTER_SEED = 20250714
PROJ_NAMES = ("qkv", "proj", "fc1", "fc2")


# --------------------------------------------------------------------------------------
# deterministic sub-seeded generators
# --------------------------------------------------------------------------------------
def rng_for(*names) -> np.random.Generator:
    """A Philox generator keyed by the master seed and a tuple of names."""
    tag = "/".join(str(n) for n in names).encode()
    h = hashlib.sha256(str(MASTER_SEED).encode() + b"|" + tag).digest()
    key = int.from_bytes(h[:8], "little")
    return np.random.Generator(np.random.Philox(key=key))


def round_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(a.shape)


def normal(shape, std, *names, mean=0.0) -> np.ndarray:
    g = rng_for(*names)
    return round_bf16((mean + std * g.standard_normal(shape)).astype(np.float32))


def uniform(shape, lo, hi, *names) -> np.ndarray:
    g = rng_for(*names)
    return round_bf16(g.uniform(lo, hi, shape).astype(np.float32))


# --------------------------------------------------------------------------------------
# containers
# --------------------------------------------------------------------------------------
@dataclass
class ModelSpec:
    img: int
    d: int
    heads: int
    mlp: int
    n_classes: int
    layers: int = 12
    patch: int = 16
    ln_eps: float = 1e-6

    @property
    def grid(self) -> int:
        return self.img // self.patch

    @property
    def tokens(self) -> int:
        return self.grid * self.grid + 1

    @property
    def patch_dim(self) -> int:
        return 3 * self.patch * self.patch

    def proj_shape(self, p: str):
        return {"qkv": (self.d, 3 * self.d), "proj": (self.d, self.d),
                "fc1": (self.d, self.mlp), "fc2": (self.mlp, self.d)}[p]


@dataclass
class Adapter:
    rank: int
    scale: float
    A: list            # [layers*4] arrays [in, rank] or None, index l*4 + {qkv,proj,fc1,fc2}
    B: list            # [layers*4] arrays [rank, out] or None
    class_ids: np.ndarray   # int32, distinct, in [0, K)
    head_w: np.ndarray      # [d, n_cls]
    head_b: np.ndarray      # [n_cls]
    acc: np.ndarray         # [n_cls] validation accuracy a_{C,l}


@dataclass
class Workload:
    name: str
    spec: ModelSpec
    backbone: dict
    adapters: list                 # list[Adapter], index = adapter id
    frames: np.ndarray             # [F, 3, img, img] float32 (bf16-representable)
    set_offsets: np.ndarray        # int32 [F+1]
    set_ids: np.ndarray            # int32 [nnz], ascending inside each frame
    tau: float = 0.6
    extra: dict = field(default_factory=dict)

    @property
    def n_frames(self) -> int:
        return int(self.frames.shape[0])

    def sets(self):
        o, i = self.set_offsets, self.set_ids
        return [list(map(int, i[o[f]:o[f + 1]])) for f in range(len(o) - 1)]


def sets_to_csr(sets):
    offsets = np.zeros(len(sets) + 1, dtype=np.int32)
    ids = []
    for f, s in enumerate(sets):
        s = sorted(set(int(a) for a in s))
        ids.extend(s)
        offsets[f + 1] = len(ids)
    return offsets, np.asarray(ids, dtype=np.int32)


# --------------------------------------------------------------------------------------
# model pieces
# --------------------------------------------------------------------------------------
def make_backbone(name: str, spec: ModelSpec, head_bias_mean: float = 0.0) -> dict:
    """Backbone weights N(0, 0.02) in row-vector convention W[in, out] (Sec. 3.1 notation)."""
    L, d, m, K, T = spec.layers, spec.d, spec.mlp, spec.n_classes, spec.tokens
    w = {}
    w["patch_w"] = normal((spec.patch_dim, d), 0.02, name, "patch_w")
    w["patch_b"] = normal((d,), 0.02, name, "patch_b")
    w["cls"] = normal((d,), 0.02, name, "cls")
    w["pos"] = normal((T, d), 0.02, name, "pos")
    w["ln1_g"] = normal((L, d), 0.02, name, "ln1_g", mean=1.0)
    w["ln1_b"] = normal((L, d), 0.02, name, "ln1_b")
    w["qkv_w"] = normal((L, d, 3 * d), 0.02, name, "qkv_w")
    w["qkv_b"] = normal((L, 3 * d), 0.02, name, "qkv_b")
    w["proj_w"] = normal((L, d, d), 0.02, name, "proj_w")
    w["proj_b"] = normal((L, d), 0.02, name, "proj_b")
    w["ln2_g"] = normal((L, d), 0.02, name, "ln2_g", mean=1.0)
    w["ln2_b"] = normal((L, d), 0.02, name, "ln2_b")
    w["fc1_w"] = normal((L, d, m), 0.02, name, "fc1_w")
    w["fc1_b"] = normal((L, m), 0.02, name, "fc1_b")
    w["fc2_w"] = normal((L, m, d), 0.02, name, "fc2_w")
    w["fc2_b"] = normal((L, d), 0.02, name, "fc2_b")
    w["lnf_g"] = normal((d,), 0.02, name, "lnf_g", mean=1.0)
    w["lnf_b"] = normal((d,), 0.02, name, "lnf_b")
    w["head_w"] = normal((d, K), 0.02, name, "head_w")
    w["head_b"] = normal((K,), 0.02, name, "head_b", mean=head_bias_mean)
    return w


def make_adapter(name: str, spec: ModelSpec, aid: int, rank: int, class_ids,
                 layers=None, projs=PROJ_NAMES, ab_std: float = 0.02) -> Adapter:
    """One LoRA adapter: A[in, r], B[r, out] per adapted (layer, projection), a head over its
    class subset and a per-class accuracy table a_{C,l} ~ U(0.5, 1).  scale = 32 / rank."""
    layers = range(spec.layers) if layers is None else layers
    A = [None] * (spec.layers * 4)
    B = [None] * (spec.layers * 4)
    for l in layers:
        for pi, p in enumerate(PROJ_NAMES):
            if p not in projs:
                continue
            kin, nout = spec.proj_shape(p)
            A[l * 4 + pi] = normal((kin, rank), ab_std, name, "A", aid, l, p)
            B[l * 4 + pi] = normal((rank, nout), ab_std, name, "B", aid, l, p)
    class_ids = np.asarray(class_ids, dtype=np.int32)
    n = len(class_ids)
    g = rng_for(name, "acc", aid)
    return Adapter(rank=rank, scale=32.0 / rank, A=A, B=B, class_ids=class_ids,
                   head_w=normal((spec.d, n), 0.02, name, "head_w", aid),
                   head_b=normal((n,), 0.02, name, "head_b", aid),
                   acc=g.uniform(0.5, 1.0, n).astype(np.float32))


def make_frames(name: str, spec: ModelSpec, n: int) -> np.ndarray:
    return uniform((n, 3, spec.img, spec.img), -1.0, 1.0, name, "frames")


def make_stream_frames(name: str, spec: ModelSpec, n_streams: int, n_steps: int,
                       noise: float = 0.05) -> np.ndarray:
    """[n_streams, n_steps, 3, img, img]: each frame = the previous one + N(0, noise)."""
    out = np.empty((n_streams, n_steps, 3, spec.img, spec.img), dtype=np.float32)
    out[:, 0] = uniform((n_streams, 3, spec.img, spec.img), -1.0, 1.0, name, "frames0")
    g = rng_for(name, "frame_noise")
    for t in range(1, n_steps):
        step = noise * g.standard_normal(out[:, 0].shape).astype(np.float32)
        out[:, t] = round_bf16(out[:, t - 1] + step)
    return out


def draw_set(g: np.random.Generator, n_adapters: int, size_probs=(0.6, 0.3, 0.1)):
    size = 1 + int(g.choice(len(size_probs), p=np.asarray(size_probs)))
    return sorted(int(a) for a in g.choice(n_adapters, size=size, replace=False))


def changing_sets(sets, n_steps: int, p: float, n_adapters: int, tag: str = ""):
    """n_steps set lists starting from `sets`: at every step each frame redraws its set with
    probability p (sizes 1/2/3 with probability 0.6/0.3/0.1, uniform distinct ids), else keeps it --
    the slowly changing sets of a video stream (temporal continuity)."""
    g = rng_for("changing_sets", tag, n_steps, p, n_adapters)
    cur = [list(s) for s in sets]
    out = []
    for _ in range(n_steps):
        cur = [draw_set(g, n_adapters) if g.random() < p else s for s in cur]
        out.append(sets_to_csr(cur))
    return out


# --------------------------------------------------------------------------------------
# the workloads
# --------------------------------------------------------------------------------------
def tiny_spec(n_classes=32, layers=12):
    return ModelSpec(img=224, d=192, heads=3, mlp=768, n_classes=n_classes, layers=layers)


def deit_tiny_2frames() -> Workload:
    """DeiT-tiny, 2 frames, 4 rank-4 adapters owning 8 classes each; sets {0} and {1,3}."""
    name = "deit_tiny_2frames"
    spec = tiny_spec(32)
    bb = make_backbone(name, spec)
    ads = [make_adapter(name, spec, a, 4, np.arange(8 * a, 8 * a + 8)) for a in range(4)]
    off, ids = sets_to_csr([[0], [1, 3]])
    return Workload(name, spec, bb, ads, make_frames(name, spec, 2), off, ids)


def deit_small_streams(n_streams=4, n_steps=16) -> Workload:
    """DeiT-small, 64 frames = 4 streams x 16 consecutive frames (stream-major), 16 rank-8
    adapters over 160 classes in disjoint groups of 10.  Each stream keeps its adapter set and
    redraws it with probability 0.1 per frame."""
    name = "deit_small_streams"
    spec = ModelSpec(img=224, d=384, heads=6, mlp=1536, n_classes=160)
    bb = make_backbone(name, spec)
    ads = [make_adapter(name, spec, a, 8, np.arange(10 * a, 10 * a + 10)) for a in range(16)]
    fr = make_stream_frames(name, spec, n_streams, n_steps)
    g = rng_for(name, "sets")
    sets = []
    for s in range(n_streams):
        cur = draw_set(g, 16)
        for t in range(n_steps):
            if t > 0 and g.random() < 0.1:
                cur = draw_set(g, 16)
            sets.append(cur)
    off, ids = sets_to_csr(sets)
    return Workload(name, spec, bb, ads, fr.reshape(-1, 3, spec.img, spec.img), off, ids)


def overlapping_groups(n_groups: int, per_group: int):
    """Partition of n_groups*per_group classes; every 10th class is also listed by the next
    group, so 10 % of classes belong to two contexts."""
    K = n_groups * per_group
    groups = [list(range(g * per_group, (g + 1) * per_group)) for g in range(n_groups)]
    for k in range(0, K, 10):
        groups[(k // per_group + 1) % n_groups].append(k)
    return K, [np.asarray(sorted(g), dtype=np.int32) for g in groups]


def vit_base_batch(n_frames=256, layers=12, lora_last=None) -> Workload:
    """ViT-base production shape: 32 rank-16 adapters over 800 classes (32 groups of 25, 10 %
    of classes shared by two groups); 60/30/10 % of frames have 1/2/3 active adapters.
    lora_last = N restricts every adapter to the last N blocks (the paper's cheap placement,
    Sec. 3.1); None adapts all blocks."""
    name = "vit_base_batch"
    spec = ModelSpec(img=224, d=768, heads=12, mlp=3072, n_classes=800, layers=layers)
    bb = make_backbone(name, spec)
    _, groups = overlapping_groups(32, 25)
    lora_layers = None if lora_last is None else range(layers - lora_last, layers)
    ads = [make_adapter(name, spec, a, 16, groups[a], layers=lora_layers) for a in range(32)]
    g = rng_for(name, "sets")
    sets = [draw_set(g, 32) for _ in range(n_frames)]
    off, ids = sets_to_csr(sets)
    return Workload(name, spec, bb, ads, make_frames(name, spec, n_frames), off, ids)


def vit_base_384_streams(n_streams=16, n_steps=30, layers=12) -> Workload:
    """ViT-base at 384x384 (577 tokens), 16 streams x 30 correlated frames, 64 rank-16 adapters
    whose class-subset sizes cycle 5/10/15/20 over a partition of 800 classes, plus 80 classes
    listed twice.  The base-head bias is shifted so that only the upper tail of the base logits
    (std ~ sqrt(d)*0.02) crosses the 0.5 score threshold: a few labels per frame."""
    name = "vit_base_384_streams"
    spec = ModelSpec(img=384, d=768, heads=12, mlp=3072, n_classes=800, layers=layers)
    logit_std = float(np.sqrt(spec.d)) * 0.02
    bb = make_backbone(name, spec, head_bias_mean=-2.807 * logit_std)
    sizes = [5, 10, 15, 20] * 16
    bounds = np.concatenate([[0], np.cumsum(sizes)])
    groups = [list(range(bounds[a], bounds[a + 1])) for a in range(64)]
    for k in range(0, 800, 10):           # 80 classes double-listed, by an adapter 7 further on
        owner = int(np.searchsorted(bounds, k, side="right") - 1)
        groups[(owner + 7) % 64].append(k)
    ads = [make_adapter(name, spec, a, 16, np.asarray(sorted(groups[a]), dtype=np.int32))
           for a in range(64)]
    fr = make_stream_frames(name, spec, n_streams, n_steps)     # [S, T, 3, 384, 384]
    off, ids = sets_to_csr([[] for _ in range(n_streams)])
    return Workload(name, spec, bb, ads, fr[:, 0].copy(), off, ids, tau=0.6,
                    extra={"stream_frames": fr, "score_thr": 0.5})


def deit_tiny_stream(n_steps=30, n_streams=1) -> Workload:
    """The paper's embedded operating point as a latency workload (Sec. 4, Table 2): DeiT-tiny, one
    video stream, 11 contexts of 5 classes each over an 80-class label space (25 classes belong to
    no context), rank-16 adapters on the query and value projections of the last 2 of 12 blocks,
    scale 32/16.  The base-head bias is shifted so that about two labels per frame cross 0.5."""
    name = "deit_tiny_stream"
    spec = tiny_spec(80)
    logit_std = float(np.sqrt(spec.d)) * 0.02
    bb = make_backbone(name, spec, head_bias_mean=-1.96 * logit_std)
    ads = []
    for a in range(11):
        ad = make_adapter(name, spec, a, 16, np.arange(5 * a, 5 * a + 5), layers=range(spec.layers - 2, spec.layers),
                          projs=("qkv",))
        for l in range(spec.layers - 2, spec.layers):
            ad.B[l * 4][:, spec.d:2 * spec.d] = 0.0          # query and value only: the key columns stay untouched
        ads.append(ad)
    fr = make_stream_frames(name, spec, n_streams, n_steps)
    off, ids = sets_to_csr([[] for _ in range(n_streams)])
    return Workload(name, spec, bb, ads, fr[:, 0].copy(), off, ids, tau=0.6,
                    extra={"stream_frames": fr, "score_thr": 0.5})


# --------------------------------------------------------------------------------------
# isolated fused base+LoRA linear cells
# --------------------------------------------------------------------------------------
@dataclass
class LinearCell:
    name: str
    k_in: int
    n_out: int
    tokens: int
    n_frames: int
    rank: int
    x: np.ndarray          # [n_frames*tokens, k_in]
    w: np.ndarray          # [k_in, n_out]
    b: np.ndarray          # [n_out]
    A: list                # per adapter [k_in, rank]
    B: list                # per adapter [rank, n_out]
    scale: float
    set_offsets: np.ndarray
    set_ids: np.ndarray


def zipf_probs(n: int, s: float = 1.2) -> np.ndarray:
    p = 1.0 / np.arange(1, n + 1) ** s
    return p / p.sum()


def linear_cell(k_in: int, n_out: int, n_frames: int, rank: int, clustered: bool,
                n_adapters: int = 128, tokens: int = 197, max_set: int = 8,
                tag: str = "") -> LinearCell:
    """One cell of the isolated linear sweep: x ~ N(0,1), W ~ N(0,0.02), 128 adapters of one
    rank, 1-8 active adapters per frame drawn uniformly or Zipf(1.2)-clustered."""
    name = f"linear_{k_in}x{n_out}_F{n_frames}_r{rank}_{'zipf' if clustered else 'unif'}{tag}"
    x = normal((n_frames * tokens, k_in), 1.0, name, "x")
    w = normal((k_in, n_out), 0.02, name, "w")
    b = normal((n_out,), 0.02, name, "b")
    A = [normal((k_in, rank), 0.02, name, "A", a) for a in range(n_adapters)]
    B = [normal((rank, n_out), 0.02, name, "B", a) for a in range(n_adapters)]
    g = rng_for(name, "sets")
    p = zipf_probs(n_adapters) if clustered else None
    sets = []
    for _ in range(n_frames):
        size = int(g.integers(1, max_set + 1))
        sets.append(sorted(int(a) for a in g.choice(n_adapters, size=size, replace=False, p=p)))
    off, ids = sets_to_csr(sets)
    return LinearCell(name, k_in, n_out, tokens, n_frames, rank, x, w, b, A, B, 32.0 / rank,
                      off, ids)


# --------------------------------------------------------------------------------------
# small random cover tables for the selection tests
# --------------------------------------------------------------------------------------
def random_cover_table(seed, n_contexts: int, n_labels: int, max_size: int, overlap: bool):
    """Contexts (sorted class-id arrays) + accuracies for selection tests.  Without overlap the
    contexts are a partition of a subset of the labels."""
    g = rng_for("cover", seed, n_contexts, n_labels, overlap)
    ctxs = []
    if overlap:
        for _ in range(n_contexts):
            sz = int(g.integers(1, max_size + 1))
            ctxs.append(np.sort(g.choice(n_labels, size=min(sz, n_labels), replace=False)).astype(np.int32))
    else:
        perm = g.permutation(n_labels)
        pos = 0
        for _ in range(n_contexts):
            sz = int(g.integers(1, max_size + 1))
            ctxs.append(np.sort(perm[pos:pos + sz]).astype(np.int32))
            pos += sz
    accs = [g.uniform(0.5, 1.0, len(c)).astype(np.float32) for c in ctxs]
    return ctxs, accs
