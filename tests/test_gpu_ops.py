"""GPU parity of the single operators (through the C ABI) against the CPU oracle."""
import numpy as np
import pytest

import workloads as wl
from oracle import polymorph_oracle as po

pytestmark = pytest.mark.gpu

# bf16 build: inputs are bf16-exact, products accumulate in fp32, the output is rounded once to
# bf16 (relative 2^-9) and the LoRA intermediate t = s (x A) once more; fp32 debug build: fp32
# accumulation order only.
TOL = {0: dict(atol=1.5e-2, rtol=1.5e-2), 1: dict(atol=2e-4, rtol=2e-4)}


def tdtype(dtype):
    import torch
    return torch.bfloat16 if dtype == 0 else torch.float32


def to_dev(a, dtype):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda().to(tdtype(dtype)).contiguous()


def to_np(t):
    return t.float().cpu().numpy().astype(np.float64)


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("rows,d", [(1, 192), (1003, 384), (2 * 197 + 5, 768), (64, 1024)])
def test_layernorm(dtype, rows, d):
    import torch
    from paper_2507_14959_b200 import binding
    x = wl.normal((rows, d), 1.0, "ln_gpu", rows, d) * 3 + 0.5
    x = wl.round_bf16(x)
    g = wl.normal((d,), 0.2, "ln_gpu_g", d, mean=1.0)
    b = wl.normal((d,), 0.2, "ln_gpu_b", d)
    xd = to_dev(x, dtype)
    yd = torch.full_like(xd, float("nan"))
    binding.layernorm(xd, torch.from_numpy(g).cuda(), torch.from_numpy(b).cuda(), yd, 1e-6, dtype)
    torch.cuda.synchronize()
    want = po.layernorm(x.astype(np.float64), g.astype(np.float64), b.astype(np.float64), 1e-6)
    np.testing.assert_allclose(to_np(yd), want, **TOL[dtype])


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("frames,tokens,heads", [(3, 197, 3), (1, 577, 2), (2, 10, 1), (2, 64, 2), (1, 130, 1),
                                                 (2, 626, 2),      # beyond the tcgen05 kernels' 624 tokens
                                                 (1, 785, 1)])     # 448x448 frames: several query slices
def test_attention(dtype, frames, tokens, heads):
    import torch
    from paper_2507_14959_b200 import binding
    d = heads * 64
    qkv = wl.normal((frames * tokens, 3 * d), 1.0, "attn_gpu", frames, tokens, heads)
    qd = to_dev(qkv, dtype)
    od = torch.full((frames * tokens, d), float("nan"), device="cuda", dtype=tdtype(dtype))
    binding.attention(qd, od, frames, tokens, heads, dtype)
    torch.cuda.synchronize()
    got = to_np(od)
    for f in range(frames):
        want = po.attention(qkv[f * tokens:(f + 1) * tokens].astype(np.float64), heads)
        np.testing.assert_allclose(got[f * tokens:(f + 1) * tokens], want, **TOL[dtype])


def test_attention_many_heads_several_query_tiles_per_cta():
    """With enough (frame, head) pairs to fill the GPU several times over, the kernel for 209..624 tokens
    gives each CTA all query tiles of its pair (instead of one tile per CTA): two key blocks and three
    query tiles here, the second and third tile reusing the score regions and O of the first.  Three
    frames of the batch are compared with the oracle."""
    import torch
    from paper_2507_14959_b200 import binding
    frames, tokens, heads = 50, 300, 12
    d = heads * 64
    qkv = wl.normal((frames * tokens, 3 * d), 1.0, "attn_gpu_many", frames, tokens, heads).astype(np.float32)
    qd = to_dev(qkv, 0)
    od = torch.full((frames * tokens, d), float("nan"), device="cuda", dtype=tdtype(0))
    binding.attention(qd, od, frames, tokens, heads, 0)
    torch.cuda.synchronize()
    got = to_np(od)
    assert np.isfinite(got).all()
    for f in (0, 17, 49):
        want = po.attention(to_np(qd[f * tokens:(f + 1) * tokens]).astype(np.float64), heads)
        np.testing.assert_allclose(got[f * tokens:(f + 1) * tokens], want, **TOL[0])


def oracle_linear(cell_x, w, b, A, B, scale, tokens, offsets, ids, epilogue, residual):
    out = np.empty((cell_x.shape[0], w.shape[1]))
    w64, b64 = w.astype(np.float64), b.astype(np.float64)
    for f in range(len(offsets) - 1):
        rows = slice(f * tokens, (f + 1) * tokens)
        act = [(scale, A[a].astype(np.float64), B[a].astype(np.float64))
               for a in sorted(ids[offsets[f]:offsets[f + 1]])]
        out[rows] = po.lora_linear(cell_x[rows].astype(np.float64), w64, b64, act)
    if epilogue == 1:
        out = po.gelu(out)
    elif epilogue == 2:
        out = out + residual
    return out


LINEAR_CASES = [
    # k_in, n_out, frames, tokens, rank, n_adapters, epilogue, sets
    (192, 576, 2, 197, 4, 4, 0, [[0], [1, 3]]),
    (192, 192, 3, 197, 4, 4, 2, [[], [2], [0, 1, 2, 3]]),
    (384, 1536, 5, 197, 8, 6, 1, [[5], [5], [0, 2], [], [1, 3, 4]]),
    (768, 2304, 5, 197, 16, 8, 0, [[0], [0, 7], [1, 2, 3], [4], [4]]),
    (3072, 768, 3, 197, 16, 4, 2, [[0, 1], [2], [3]]),
    (768, 3072, 2, 577, 32, 5, 1, [[0, 4], [1, 2, 3]]),
    (768, 768, 3, 197, 64, 9, 0, [[0, 1, 2, 3, 4, 5, 6, 7], [8], [2, 8]]),
    (128, 256, 7, 10, 16, 3, 0, [[0], [1], [2], [0, 1], [], [1, 2], [0, 1, 2]]),   # many frames per tile
    (768, 2304, 4, 197, 16, 2, 0, [[], [], [], []]),                                # no LoRA at all
]


@pytest.mark.parametrize("dtype", [0, 1])
@pytest.mark.parametrize("case", LINEAR_CASES, ids=[f"{c[0]}x{c[1]}_F{c[2]}_T{c[3]}_r{c[4]}_e{c[6]}" for c in LINEAR_CASES])
def test_lora_linear(dtype, case):
    import torch
    from paper_2507_14959_b200 import binding
    k_in, n_out, frames, tokens, rank, n_ad, epi, sets = case
    name = f"lin_gpu_{k_in}_{n_out}_{rank}"
    rows = frames * tokens
    x = wl.normal((rows, k_in), 1.0, name, "x")
    w = wl.normal((k_in, n_out), 0.02, name, "w")
    b = wl.normal((n_out,), 0.02, name, "b")
    A = [wl.normal((k_in, rank), 0.02, name, "A", a) for a in range(n_ad)]
    B = [wl.normal((rank, n_out), 0.02, name, "B", a) for a in range(n_ad)]
    res = wl.normal((rows, n_out), 1.0, name, "res")
    scale = 32.0 / rank
    off, ids = wl.sets_to_csr(sets)
    max_set = max(1, max(len(s) for s in sets))
    lin = binding.Linear(w, b, max_adapters=n_ad, max_rank=rank, max_set=max_set, max_frames=frames,
                         tokens=tokens, epilogue=epi, dtype=dtype)
    for a in range(n_ad):
        lin.register(a, rank, scale, A[a], B[a])
    xd = to_dev(x, dtype)
    rd = to_dev(res, dtype) if epi == 2 else None
    yd = torch.full((rows, n_out), float("nan"), device="cuda", dtype=tdtype(dtype))
    lin.forward(xd, frames, off, ids, yd, residual=rd)
    assert lin.status() == 0
    got = to_np(yd)
    want = oracle_linear(x, w, b, A, B, scale, tokens, off, ids, epi, res.astype(np.float64))
    np.testing.assert_allclose(got, want, **TOL[dtype])
    # a second call with the same sets reuses the cached plan and must give the same bits
    y2 = torch.full_like(yd, float("nan"))
    lin.forward(xd, frames, off, ids, y2, residual=rd)
    assert lin.status() == 0
    assert torch.equal(yd, y2)
    # LoRA really contributes where a set is non-empty
    if any(sets):
        base = oracle_linear(x, w, b, A, B, scale, tokens, np.zeros(frames + 1, np.int32), ids[:0], epi,
                             res.astype(np.float64))
        assert np.abs(want - base).max() > 0.05
    lin.close()


FULL_SIZE_CELLS = [
    # k_in, n_out, rank, clustered, epilogue
    (768, 2304, 16, False, 0),
    (3072, 768, 64, False, 2),      # rank 64 with up to 8 active adapters: the largest LoRA share
    (768, 3072, 64, False, 1),
    (768, 2304, 32, True, 0),       # Zipf-clustered sets
    (3072, 768, 8, True, 2),        # rank below one slab
]


@pytest.mark.parametrize("k_in,n_out,rank,clustered,epi", FULL_SIZE_CELLS,
                         ids=[f"{c[0]}x{c[1]}_r{c[2]}_{'zipf' if c[3] else 'unif'}_e{c[4]}" for c in FULL_SIZE_CELLS])
def test_lora_linear_full_size_sampled(k_in, n_out, rank, clustered, epi):
    """Cells of the single-linear grid at full size (256 frames x 197 tokens, 128 adapters of one
    rank, 1-8 active per frame) in the launch configuration the sweep times; the oracle computes
    sampled rows one by one: first and last row tiles, frame boundaries, the ragged tail, rows of
    the frames with the most active adapters, and random rows."""
    import torch
    from paper_2507_14959_b200 import binding
    cell = wl.linear_cell(k_in, n_out, 256, rank, clustered=clustered)
    lin = binding.Linear(cell.w, cell.b, max_adapters=128, max_rank=rank, max_set=8, max_frames=256,
                         tokens=cell.tokens, epilogue=epi, dtype=0)
    for a in range(128):
        lin.register(a, rank, cell.scale, cell.A[a], cell.B[a])
    rows = 256 * cell.tokens
    xd = to_dev(cell.x, 0)
    res = wl.normal((rows, n_out), 1.0, cell.name, "res") if epi == 2 else None
    rd = to_dev(res, 0) if epi == 2 else None
    yd = torch.full((rows, n_out), float("nan"), device="cuda", dtype=torch.bfloat16)
    lin.forward(xd, 256, cell.set_offsets, cell.set_ids, yd, residual=rd)
    assert lin.status() == 0
    assert not torch.isnan(yd.float()).any()
    g = wl.rng_for("full_size_rows", k_in, n_out, rank)
    sizes = np.diff(cell.set_offsets)
    assert sizes.max() == 8
    widest = [int(f) for f in np.argsort(-sizes, kind="stable")[:3]]
    sample = sorted(set([0, 127, 128, 196, 197, 198, rows - 1, rows - 65, rows - 128, rows - 129]
                        + [f * cell.tokens + t for f in widest for t in (0, 100, 196)]
                        + [int(r) for r in g.integers(0, rows, 48)]))
    got = to_np(yd[sample])
    w64, b64 = cell.w.astype(np.float64), cell.b.astype(np.float64)
    for i, r in enumerate(sample):
        f = r // cell.tokens
        act = [(cell.scale, cell.A[a].astype(np.float64), cell.B[a].astype(np.float64))
               for a in sorted(cell.set_ids[cell.set_offsets[f]:cell.set_offsets[f + 1]])]
        want = po.lora_linear(cell.x[r:r + 1].astype(np.float64), w64, b64, act)[0]
        if epi == 1:
            want = po.gelu(want)
        elif epi == 2:
            want = want + wl.round_bf16(res[r]).astype(np.float64)
        np.testing.assert_allclose(got[i], want, **TOL[0])
    lin.close()


def test_gelu_epilogue_accuracy():
    """The GELU epilogue against the exact-erf definition: y = gelu(4 x) through an identity-like
    weight, x sweeping [-3, 3] (so the argument spans [-12, 12]); the bf16 result must be within one
    bf16 step of the exact value plus 3e-5 (the kernel evaluates a fitted form x (1/2 + 1/2 tanh(x q(x^2)))
    of x Phi(x) whose absolute error stays below 2.6e-5, with the hardware's approximate tanh)."""
    import torch
    from paper_2507_14959_b200 import binding
    n, rows = 64, 197 * 3
    w = 4.0 * np.eye(n, dtype=np.float32)
    x = wl.round_bf16(np.linspace(-3.0, 3.0, rows * n, dtype=np.float32).reshape(rows, n))
    lin = binding.Linear(w, np.zeros(n, np.float32), max_adapters=1, max_rank=16, max_set=1, max_frames=3,
                         tokens=197, epilogue=1, dtype=0)
    xd = to_dev(x, 0)
    yd = torch.full((rows, n), float("nan"), device="cuda", dtype=torch.bfloat16)
    lin.forward(xd, 3, np.zeros(4, np.int32), np.zeros(0, np.int32), yd)
    assert lin.status() == 0
    want = po.gelu(4.0 * x.astype(np.float64))
    got = to_np(yd)
    step = np.maximum(np.abs(want), 2.0 ** -20) * 2.0 ** -8          # one bf16 step at |want|
    assert np.all(np.abs(got - want) <= step + 3e-5)
    assert np.all(got[want > 11.0] == wl.round_bf16(want[want > 11.0].astype(np.float32)))   # saturated branch: x itself
    lin.close()


def test_linear_argument_errors():
    import torch
    from paper_2507_14959_b200 import binding
    w = wl.normal((64, 64), 0.02, "err_w")
    b = np.zeros(64, np.float32)
    lin = binding.Linear(w, b, max_adapters=2, max_rank=16, max_set=1, max_frames=2, tokens=8, dtype=0)
    lin.register(0, 16, 2.0, np.zeros((64, 16), np.float32), np.zeros((16, 64), np.float32))
    x = torch.zeros((16, 64), device="cuda", dtype=torch.bfloat16)
    y = torch.zeros_like(x)
    with pytest.raises(binding.PolymorphError) as e:      # unregistered adapter
        lin.forward(x, 2, [0, 1, 2], [0, 1], y)
    assert e.value.code == binding.PM_ERR_STATE
    with pytest.raises(binding.PolymorphError) as e:      # set larger than max_set
        lin.forward(x, 2, [0, 2, 2], [0, 0], y)
    assert e.value.code == binding.PM_ERR_CAPACITY
    with pytest.raises(binding.PolymorphError) as e:      # non-monotone CSR
        lin.forward(x, 2, [0, 1, 0], [0], y)
    assert e.value.code == binding.PM_ERR_ARG
    with pytest.raises(binding.PolymorphError) as e:      # too many frames
        lin.forward(x, 3, [0, 0, 0, 0], [], y)
    assert e.value.code == binding.PM_ERR_CAPACITY
    with pytest.raises(binding.PolymorphError) as e:      # rank above max_rank
        lin.register(1, 32, 1.0, np.zeros((64, 32), np.float32), np.zeros((32, 64), np.float32))
    assert e.value.code == binding.PM_ERR_CAPACITY
    lin.close()


def test_bounded_wait_gives_up_and_reports():
    """A wait on a barrier that nothing signals runs into its limit, records PM_ERR_TIMEOUT, takes the
    other warps of the CTA out through the abort flag and releases tensor memory; nothing faults and
    the next kernel on the device runs normally."""
    import torch
    from paper_2507_14959_b200 import binding
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    trace = torch.full((3,), -1, dtype=torch.int32, device="cuda")
    binding.selftest_wait_timeout(100000, status, trace)
    torch.cuda.synchronize()
    assert int(status.item()) == binding.PM_ERR_TIMEOUT
    assert trace.cpu().tolist() == [1, 3, 1]
    # the context is intact: an ordinary operator right after
    x = wl.normal((64, 128), 1.0, "after_timeout")
    y = torch.zeros((64, 128), device="cuda")
    binding.layernorm(torch.from_numpy(x).cuda(), torch.ones(128, device="cuda"), torch.zeros(128, device="cuda"),
                      y, 1e-6, 1)
    torch.cuda.synchronize()
    np.testing.assert_allclose(y.cpu().numpy(), po.layernorm(x.astype(np.float64), np.ones(128), np.zeros(128), 1e-6),
                               atol=2e-4)
    with pytest.raises(binding.PolymorphError):
        binding.selftest_wait_timeout(10 ** 12, status, trace)       # limits beyond 1e8 cycles are refused
