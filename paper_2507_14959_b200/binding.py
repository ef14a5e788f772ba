"""ctypes binding of libpolymorph.so: argument marshalling only.

Every function mirrors the C entry point of the same name (include/polymorph.h).  Device buffers
are torch CUDA tensors (torch is used for device memory and streams, nothing else); model
weights are numpy float32 arrays on the host.  There is no CPU fallback: if the shared library
is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes as C
import os

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpolymorph.so")

PM_OK, PM_ERR_ARG, PM_ERR_STATE, PM_ERR_CAPACITY, PM_ERR_CUDA, PM_ERR_TIMEOUT, PM_ERR_OOM = 0, -1, -2, -3, -4, -5, -6
ERROR_NAMES = {0: "PM_OK", -1: "PM_ERR_ARG", -2: "PM_ERR_STATE", -3: "PM_ERR_CAPACITY",
               -4: "PM_ERR_CUDA", -5: "PM_ERR_TIMEOUT", -6: "PM_ERR_OOM"}

EXPORTS = [
    "pm_create", "pm_register_adapter", "pm_set_cover", "pm_destroy", "pm_forward", "pm_forward_branched", "pm_forward_device_sets", "pm_select",
    "pm_select_static", "pm_metrics_reset", "pm_metrics_read", "pm_status", "pm_last_error", "pm_launch_count", "pm_set_graphs", "pm_set_small_batch_kernel", "pm_profile_enable", "pm_profile_read", "pm_plan_stats", "pm_linear_create", "pm_linear_register",
    "pm_linear_forward", "pm_linear_status", "pm_linear_last_error", "pm_linear_destroy",
    "pm_layernorm", "pm_attention", "pm_selftest_wait_timeout", "pm_cooccurrence", "pm_build_contexts", "pm_intra_coherence",
]


class PolymorphError(RuntimeError):
    def __init__(self, code, where, detail=""):
        self.code = code
        super().__init__(f"{where}: {ERROR_NAMES.get(code, code)} {detail}".strip())


class pm_config(C.Structure):
    _fields_ = [("img", C.c_int), ("patch", C.c_int), ("d", C.c_int), ("layers", C.c_int),
                ("heads", C.c_int), ("mlp", C.c_int), ("n_classes", C.c_int), ("ln_eps", C.c_float),
                ("max_adapters", C.c_int), ("max_rank", C.c_int), ("max_set", C.c_int),
                ("max_frames", C.c_int), ("dtype", C.c_int)]


_FP = C.POINTER(C.c_float)
BACKBONE_FIELDS = ["patch_w", "patch_b", "cls", "pos", "ln1_g", "ln1_b", "qkv_w", "qkv_b", "proj_w",
                   "proj_b", "ln2_g", "ln2_b", "fc1_w", "fc1_b", "fc2_w", "fc2_b", "lnf_g", "lnf_b",
                   "head_w", "head_b"]


class pm_backbone(C.Structure):
    _fields_ = [(n, _FP) for n in BACKBONE_FIELDS]


class pm_adapter(C.Structure):
    _fields_ = [("rank", C.c_int), ("scale", C.c_float), ("A", C.POINTER(_FP)), ("B", C.POINTER(_FP)),
                ("n_cls", C.c_int), ("class_ids", C.POINTER(C.c_int32)), ("head_w", _FP),
                ("head_b", _FP), ("acc", _FP)]


_lib = None


def load():
    """Loads the shared library (building nothing).  Raises if it is not there."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2507_14959_b200.build` "
                           "(there is no fallback path)")
    lib = C.CDLL(LIB_PATH)
    vp, ip = C.c_void_p, C.c_int
    lib.pm_create.argtypes = [C.POINTER(pm_config), C.POINTER(pm_backbone), C.POINTER(vp)]
    lib.pm_register_adapter.argtypes = [vp, ip, C.POINTER(pm_adapter)]
    lib.pm_set_cover.argtypes = [vp, C.c_float]
    lib.pm_destroy.argtypes = [vp]
    lib.pm_destroy.restype = None
    lib.pm_forward.argtypes = [vp, vp, ip, vp, vp, vp, vp, vp]
    lib.pm_forward_device_sets.argtypes = [vp, vp, ip, vp, vp, vp, vp, vp]
    lib.pm_forward_branched.argtypes = [vp, vp, ip, vp, vp, ip, vp, vp, vp]
    lib.pm_select.argtypes = [vp, vp, ip, C.c_float, ip, ip, vp, vp, vp, vp, vp, ip, vp]
    lib.pm_select_static.argtypes = [vp, ip, ip, ip, C.c_float, ip, ip, vp, vp, vp, vp, vp, vp, vp, ip, vp, vp]
    lib.pm_status.argtypes = [vp, vp]
    lib.pm_metrics_reset.argtypes = [vp, vp]
    lib.pm_metrics_read.argtypes = [vp, vp, C.POINTER(C.c_longlong), C.POINTER(C.c_longlong), C.POINTER(C.c_longlong)]
    lib.pm_last_error.argtypes = [vp]
    lib.pm_last_error.restype = C.c_char_p
    lib.pm_launch_count.argtypes = [vp]
    lib.pm_cooccurrence.argtypes = [vp, ip, ip, vp, vp, vp]
    lib.pm_build_contexts.argtypes = [_FP, ip, ip, ip, ip, C.POINTER(C.c_int32), C.POINTER(C.c_int32), C.POINTER(C.c_int)]
    lib.pm_intra_coherence.argtypes = [_FP, ip, C.POINTER(C.c_int32), C.POINTER(C.c_int32), ip, C.POINTER(C.c_double)]
    lib.pm_set_graphs.argtypes = [vp, ip]
    lib.pm_set_small_batch_kernel.argtypes = [vp, ip]
    lib.pm_launch_count.restype = C.c_longlong
    lib.pm_profile_enable.argtypes = [vp, ip]
    lib.pm_profile_read.argtypes = [vp, vp, C.POINTER(C.c_double), C.POINTER(C.c_longlong)]
    lib.pm_plan_stats.argtypes = [vp, C.POINTER(C.c_longlong), C.POINTER(C.c_double)]
    lib.pm_linear_create.argtypes = [ip, ip, _FP, _FP, ip, ip, ip, ip, ip, ip, ip, C.POINTER(vp)]
    lib.pm_linear_register.argtypes = [vp, ip, ip, C.c_float, _FP, _FP]
    lib.pm_linear_forward.argtypes = [vp, vp, ip, vp, vp, vp, vp, vp]
    lib.pm_linear_status.argtypes = [vp, vp]
    lib.pm_linear_last_error.argtypes = [vp]
    lib.pm_linear_last_error.restype = C.c_char_p
    lib.pm_linear_destroy.argtypes = [vp]
    lib.pm_linear_destroy.restype = None
    lib.pm_layernorm.argtypes = [vp, vp, vp, vp, ip, ip, C.c_float, ip, vp]
    lib.pm_attention.argtypes = [vp, vp, ip, ip, ip, ip, vp]
    lib.pm_selftest_wait_timeout.argtypes = [C.c_longlong, vp, vp, vp]
    _lib = lib
    return lib


def _f32(a):
    return np.ascontiguousarray(a, dtype=np.float32)


def _fp(a):
    return a.ctypes.data_as(_FP)


def _ptr(t):
    """Address of a torch tensor / numpy array / None as a void pointer value."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream_ptr(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


class Model:
    """Owner of a pm_handle.  Methods are the C calls with the handle bound."""

    def __init__(self, *, img, d, layers, heads, mlp, n_classes, backbone, max_adapters, max_rank,
                 max_set, max_frames, dtype=0, patch=16, ln_eps=1e-6):
        lib = load()
        self.lib = lib
        self.cfg = pm_config(img, patch, d, layers, heads, mlp, n_classes, ln_eps, max_adapters,
                             max_rank, max_set, max_frames, dtype)
        keep = {k: _f32(backbone[k]) for k in BACKBONE_FIELDS}
        bb = pm_backbone(**{k: _fp(v) for k, v in keep.items()})
        self.handle = C.c_void_p()
        rc = lib.pm_create(C.byref(self.cfg), C.byref(bb), C.byref(self.handle))
        if rc != PM_OK:
            self.handle = None
            raise PolymorphError(rc, "pm_create")
        self.n_classes = n_classes
        self.dtype = dtype

    def _check(self, rc, where):
        if rc != PM_OK:
            raise PolymorphError(rc, where, self.lib.pm_last_error(self.handle).decode())

    def register_adapter(self, adapter_id, *, rank, scale, A, B, class_ids, head_w, head_b, acc=None):
        n = len(A)
        keepA = [None if m is None else _f32(m) for m in A]
        keepB = [None if m is None else _f32(m) for m in B]
        arrA = (_FP * n)(*[None if m is None else _fp(m) for m in keepA])
        arrB = (_FP * n)(*[None if m is None else _fp(m) for m in keepB])
        cls = np.ascontiguousarray(class_ids, dtype=np.int32)
        hw, hb = _f32(head_w), _f32(head_b)
        ac = None if acc is None else _f32(acc)
        ad = pm_adapter(rank, scale, arrA, arrB, len(cls), cls.ctypes.data_as(C.POINTER(C.c_int32)),
                        _fp(hw), _fp(hb), None if ac is None else _fp(ac))
        self._check(self.lib.pm_register_adapter(self.handle, adapter_id, C.byref(ad)), "pm_register_adapter")

    def set_cover(self, tau):
        self._check(self.lib.pm_set_cover(self.handle, tau), "pm_set_cover")

    def forward(self, frames, set_offsets, set_ids, scores_out, base_out=None, stream=None):
        """frames/scores_out/base_out: torch CUDA tensors; set lists: numpy int32 (host) or torch
        CUDA int32 tensors."""
        n = int(frames.shape[0])
        if isinstance(set_offsets, np.ndarray):
            set_offsets = np.ascontiguousarray(set_offsets, dtype=np.int32)
        if isinstance(set_ids, np.ndarray):
            set_ids = np.ascontiguousarray(set_ids, dtype=np.int32)
        self._check(self.lib.pm_forward(self.handle, _ptr(frames), n, _ptr(set_offsets), _ptr(set_ids),
                                        _ptr(scores_out), _ptr(base_out), _stream_ptr(stream)), "pm_forward")

    def forward_device_sets(self, frames, set_offsets, set_ids, scores_out, base_out=None, stream=None):
        """pm_forward_device_sets: the set lists are torch CUDA int32 tensors (e.g. written by
        select()); the plan is built on the device, nothing synchronises."""
        self._check(self.lib.pm_forward_device_sets(self.handle, _ptr(frames), int(frames.shape[0]),
                                                    _ptr(set_offsets), _ptr(set_ids), _ptr(scores_out),
                                                    _ptr(base_out), _stream_ptr(stream)), "pm_forward_device_sets")

    def forward_branched(self, frames, set_offsets, set_ids, trunk_layers, scores_out, base_out=None, stream=None):
        """pm_forward_branched: shared trunk of `trunk_layers` blocks, then one branch per active
        adapter (and the base branch if base_out is given).  Arguments as for forward()."""
        n = int(frames.shape[0])
        if isinstance(set_offsets, np.ndarray):
            set_offsets = np.ascontiguousarray(set_offsets, dtype=np.int32)
        if isinstance(set_ids, np.ndarray):
            set_ids = np.ascontiguousarray(set_ids, dtype=np.int32)
        self._check(self.lib.pm_forward_branched(self.handle, _ptr(frames), n, _ptr(set_offsets), _ptr(set_ids),
                                                 int(trunk_layers), _ptr(scores_out), _ptr(base_out),
                                                 _stream_ptr(stream)), "pm_forward_branched")

    def select(self, scores, score_thr, context_copy, has_prev, prev_labels, prev_offsets, prev_ids,
               next_offsets, next_ids, stream=None):
        n = int(scores.shape[0])
        cap = 0 if next_ids is None else int(next_ids.numel())
        self._check(self.lib.pm_select(self.handle, _ptr(scores), n, score_thr, int(context_copy),
                                       int(has_prev), _ptr(prev_labels), _ptr(prev_offsets), _ptr(prev_ids),
                                       _ptr(next_offsets), _ptr(next_ids), cap, _stream_ptr(stream)), "pm_select")

    def status(self, stream=None):
        return self.lib.pm_status(self.handle, _stream_ptr(stream))

    def metrics_reset(self, stream=None):
        self._check(self.lib.pm_metrics_reset(self.handle, _stream_ptr(stream)), "pm_metrics_reset")

    def metrics_read(self, stream=None):
        """(frames, contexts, switches) counted by select() since the last reset; synchronises."""
        f, c, s = C.c_longlong(0), C.c_longlong(0), C.c_longlong(0)
        self._check(self.lib.pm_metrics_read(self.handle, _stream_ptr(stream), C.byref(f), C.byref(c), C.byref(s)),
                    "pm_metrics_read")
        return int(f.value), int(c.value), int(s.value)

    def set_graphs(self, on):
        """Switches the recording / replaying of the forward's launch sequence as CUDA graphs."""
        self._check(self.lib.pm_set_graphs(self.handle, int(on)), "pm_set_graphs")

    def set_small_batch_kernel(self, on):
        """Whether small batches of small models run as the one whole-network kernel (default on)."""
        self._check(self.lib.pm_set_small_batch_kernel(self.handle, int(on)), "pm_set_small_batch_kernel")

    KERNEL_CLASSES = ("gemm", "shrink", "attention", "layernorm", "other", "heads", "select", "plan")

    def profile_enable(self, on):
        self._check(self.lib.pm_profile_enable(self.handle, int(on)), "pm_profile_enable")

    def profile_read(self, stream=None):
        """{class: (total_ms, launch_sites)} since the last read; synchronises the stream."""
        ms = (C.c_double * len(self.KERNEL_CLASSES))()
        n = (C.c_longlong * len(self.KERNEL_CLASSES))()
        self._check(self.lib.pm_profile_read(self.handle, _stream_ptr(stream), ms, n), "pm_profile_read")
        return {k: (ms[i], int(n[i])) for i, k in enumerate(self.KERNEL_CLASSES)}

    def plan_stats(self):
        """(plans built on the host, total host milliseconds spent building them)."""
        n, ms = C.c_longlong(0), C.c_double(0.0)
        self._check(self.lib.pm_plan_stats(self.handle, C.byref(n), C.byref(ms)), "pm_plan_stats")
        return int(n.value), float(ms.value)

    def launch_count(self):
        return int(self.lib.pm_launch_count(self.handle))

    def close(self):
        if getattr(self, "handle", None):
            self.lib.pm_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


class Linear:
    """Owner of a pm_linear (one isolated base + multi-LoRA linear)."""

    def __init__(self, w, bias, *, max_adapters, max_rank, max_set, max_frames, tokens, epilogue=0, dtype=0):
        lib = load()
        self.lib = lib
        w, bias = _f32(w), _f32(bias)
        self.k_in, self.n_out = w.shape
        self.tokens = tokens
        self.handle = C.c_void_p()
        rc = lib.pm_linear_create(self.k_in, self.n_out, _fp(w), _fp(bias), max_adapters, max_rank, max_set,
                                  max_frames, tokens, epilogue, dtype, C.byref(self.handle))
        if rc != PM_OK:
            self.handle = None
            raise PolymorphError(rc, "pm_linear_create")

    def _check(self, rc, where):
        if rc != PM_OK:
            raise PolymorphError(rc, where, self.lib.pm_linear_last_error(self.handle).decode())

    def register(self, adapter_id, rank, scale, A, B):
        A, B = _f32(A), _f32(B)
        self._check(self.lib.pm_linear_register(self.handle, adapter_id, rank, scale, _fp(A), _fp(B)),
                    "pm_linear_register")

    def forward(self, x, n_frames, set_offsets, set_ids, y, residual=None, stream=None):
        so = np.ascontiguousarray(set_offsets, dtype=np.int32)
        si = np.ascontiguousarray(set_ids, dtype=np.int32)
        self._check(self.lib.pm_linear_forward(self.handle, _ptr(x), n_frames, _ptr(so), _ptr(si),
                                               _ptr(residual), _ptr(y), _stream_ptr(stream)), "pm_linear_forward")

    def status(self, stream=None):
        return self.lib.pm_linear_status(self.handle, _stream_ptr(stream))

    def close(self):
        if getattr(self, "handle", None):
            self.lib.pm_linear_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def layernorm(x, gamma, beta, y, eps, dtype, stream=None):
    rc = load().pm_layernorm(_ptr(x), _ptr(gamma), _ptr(beta), _ptr(y), int(x.shape[0]), int(x.shape[1]),
                             eps, dtype, _stream_ptr(stream))
    if rc != PM_OK:
        raise PolymorphError(rc, "pm_layernorm")


def attention(qkv, out, n_frames, tokens, heads, dtype, stream=None):
    rc = load().pm_attention(_ptr(qkv), _ptr(out), n_frames, tokens, heads, dtype, _stream_ptr(stream))
    if rc != PM_OK:
        raise PolymorphError(rc, "pm_attention")


def selftest_wait_timeout(limit_cycles, status, trace, stream=None):
    """pm_selftest_wait_timeout: status = torch CUDA int32 [1], trace = torch CUDA int32 [3]."""
    rc = load().pm_selftest_wait_timeout(int(limit_cycles), _ptr(status), _ptr(trace), _stream_ptr(stream))
    if rc != PM_OK:
        raise PolymorphError(rc, "pm_selftest_wait_timeout")


def select_static(scores, n_adapters, score_thr, context_copy, has_prev, prev_labels, prev_offsets, prev_ids,
                  first, provider, next_offsets, next_ids, status_out=None, stream=None):
    """pm_select_static: Algorithm 2 with caller-provided cover tables and no device allocation."""
    n, k = int(scores.shape[0]), int(scores.shape[1])
    cap = 0 if next_ids is None else int(next_ids.numel())
    rc = load().pm_select_static(_ptr(scores), n, k, int(n_adapters), score_thr, int(context_copy), int(has_prev),
                                 _ptr(prev_labels), _ptr(prev_offsets), _ptr(prev_ids), _ptr(first),
                                 _ptr(provider), _ptr(next_offsets), _ptr(next_ids), cap, _ptr(status_out),
                                 _stream_ptr(stream))
    if rc != PM_OK:
        raise PolymorphError(rc, "pm_select_static")


def model_from_workload(w, *, dtype=0, max_frames=None, max_set=None):
    """Builds a Model from a workloads.Workload-shaped object (duck-typed: .spec, .backbone,
    .adapters) and registers all its adapters."""
    spec = w.spec
    ads = w.adapters
    if max_set is None:
        sizes = np.diff(w.set_offsets)
        max_set = max(3, int(sizes.max()) if len(sizes) else 0)
    m = Model(img=spec.img, d=spec.d, layers=spec.layers, heads=spec.heads, mlp=spec.mlp,
              n_classes=spec.n_classes, backbone=w.backbone, max_adapters=max(1, len(ads)),
              max_rank=max([a.rank for a in ads] + [1]), max_set=max_set,
              max_frames=max_frames or max(1, int(w.frames.shape[0])), dtype=dtype, patch=spec.patch,
              ln_eps=spec.ln_eps)
    for i, a in enumerate(ads):
        m.register_adapter(i, rank=a.rank, scale=a.scale, A=a.A, B=a.B, class_ids=a.class_ids,
                           head_w=a.head_w, head_b=a.head_b, acc=a.acc)
    return m


def cooccurrence(labels, n_labels, co, status=None, stream=None):
    """pm_cooccurrence: labels = torch CUDA int32 [T, ceil(K/32)] bit sets, co = torch CUDA fp32 [K, K]."""
    rc = load().pm_cooccurrence(_ptr(labels), int(labels.shape[0]), int(n_labels), _ptr(co), _ptr(status),
                                _stream_ptr(stream))
    if rc != PM_OK:
        raise PolymorphError(rc, "pm_cooccurrence")


def build_contexts(co, max_size, max_contexts, allow_overlap):
    """pm_build_contexts (Algorithm 1) on a host matrix; returns the contexts as lists of label ids."""
    co = np.ascontiguousarray(co, dtype=np.float32)
    K = co.shape[0]
    off = np.zeros(max_contexts + 1, dtype=np.int32)
    ids = np.zeros(max_contexts * max_size, dtype=np.int32)
    n = C.c_int(0)
    i32 = C.POINTER(C.c_int32)
    rc = load().pm_build_contexts(co.ctypes.data_as(_FP), K, int(max_size), int(max_contexts), int(bool(allow_overlap)),
                                  off.ctypes.data_as(i32), ids.ctypes.data_as(i32), C.byref(n))
    if rc != PM_OK:
        raise PolymorphError(rc, "pm_build_contexts")
    return [ids[off[c]:off[c + 1]].tolist() for c in range(n.value)]


def intra_coherence(contexts, co_norm):
    """pm_intra_coherence (Eq. 6)."""
    co_norm = np.ascontiguousarray(co_norm, dtype=np.float32)
    off, ids = [0], []
    for c in contexts:
        ids.extend(int(i) for i in c)
        off.append(len(ids))
    off = np.asarray(off, dtype=np.int32)
    ids = np.asarray(ids if ids else [0], dtype=np.int32)
    out = C.c_double(0.0)
    i32 = C.POINTER(C.c_int32)
    rc = load().pm_intra_coherence(co_norm.ctypes.data_as(_FP), co_norm.shape[0], off.ctypes.data_as(i32),
                                   ids.ctypes.data_as(i32), len(contexts), C.byref(out))
    if rc != PM_OK:
        raise PolymorphError(rc, "pm_intra_coherence")
    return out.value
