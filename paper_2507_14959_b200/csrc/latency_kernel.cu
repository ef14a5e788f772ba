// Whole-network kernel for a handful of frames (the single-stream operating point of Sec. 4): patch
// embedding, all encoder blocks with their unmerged LoRA terms (Sec. 3.1), final LayerNorm, base and
// adapter heads with sigmoid and merge (Fig. 5b) in ONE launch.
//
// Everything in a ViT block except attention is local to a token row, so a CTA owns 16 token rows of one
// frame from the first layer to the last and keeps their residual stream (fp32) and every intermediate in
// shared memory; the weights stream through a ring of 16 KB shared-memory slots filled by TMA (one
// [128 outputs x 64 inputs] box per slot, 128B swizzle, several boxes in flight) and are the only thing
// read from L2 -- every CTA reads all of them, which is what bounds a frame's latency.  The one exchange
// per block is attention: each CTA publishes the keys and values of its rows (two global buffers used in
// turn), the CTAs of a frame meet at a counter (bounded wait), then each CTA attends from its 16 query rows
// to all keys of its frame, head by head (the eight warps split the keys and merge their partial softmax
// results).  Contractions run on mma.sync m16n8k16 (bf16 in, fp32 accumulate; measured 2048 FLOP per clock
// per SM on B200, a quarter of the tcgen05 rate): with 16 rows per CTA there is no 128-row tile to give to
// tcgen05, and the tensor work is a small part of the time anyway.  What bounds a frame is that each of the
// 13 CTAs streams every weight through one SM's path to L2.
// LayerNorm uses the folded form the other kernels use: y = rstd (x W' - mean g) + b'.
#include "common.cuh"

#define BUMP(L) do { if ((L).launches) ++*(L).launches; } while (0)

namespace {

constexpr int LT_ROWS = 16;
constexpr int LT_THREADS = 256;
constexpr int LT_WARPS = 8;
constexpr int LT_GROUP = 3;                // K boxes multiplied between two CTA-wide barriers
constexpr int LT_SLOTS = 2 * LT_GROUP;     // weight ring: two groups of boxes
constexpr int LT_BOX_BYTES = 128 * 128;    // [128 output rows][64 bf16 inputs], 128B swizzle
constexpr int LT_MAX_SET = 8;
constexpr int LT_HD = 64;
constexpr long long LT_WAIT_CYCLES = 4000000000ll;

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm2(uint32_t addr, uint32_t& r0, uint32_t& r1) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}
__device__ __forceinline__ void ldsm4t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma16816(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pk_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void cp16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t bar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
__device__ __forceinline__ void tma_box(uint32_t dst, const CUtensorMap* tm, int x, int y, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(tm), "r"(x), "r"(y), "r"(bar) : "memory");
}

}  // namespace

namespace {

struct LatSmem {               // offsets (bytes) into dynamic shared memory
    int region, xres, abuf, hbuf, qbuf, tbuf, stats, part, misc, total;
    int lda, ldh, ldq, ldt;    // row strides in bf16 elements
    int kv_head;               // bytes of one head's keys + values in the region
};

__host__ __device__ inline LatSmem lat_layout(int d, int mlp, int patch_dim, int rs_total, int tokens) {
    LatSmem s;
    auto up = [](int v) { return (v + 127) & ~127; };
    s.lda = d + 8; s.ldh = (mlp > patch_dim ? mlp : patch_dim) + 8; s.ldq = d + 8; s.ldt = rs_total + 8;
    // first (1024-byte aligned, as the 128B swizzle wants): the weight ring, or two heads' keys and values
    // (each [tpad rows][128 bytes]) -- the next head's land while this one is computed
    const int tpad = (tokens + 15) / 16 * 16;
    s.kv_head = 2 * ((tpad * 128 + 1023) & ~1023);
    const int wbytes = LT_SLOTS * LT_BOX_BYTES, kvbytes = 2 * s.kv_head;
    int o = 0;
    s.region = o; o = up(o + (wbytes > kvbytes ? wbytes : kvbytes));
    s.xres = o; o = up(o + LT_ROWS * d * 4);
    s.abuf = o; o = up(o + LT_ROWS * s.lda * 2);
    s.hbuf = o; o = up(o + LT_ROWS * s.ldh * 2);
    s.qbuf = o; o = up(o + LT_ROWS * s.ldq * 2);
    s.tbuf = o; o = up(o + LT_ROWS * s.ldt * 2);
    s.stats = o; o = up(o + LT_ROWS * 16);
    s.part = o; o = up(o + LT_WARPS * LT_ROWS * (LT_HD + 2) * 4);      // partial attention results of the warps
    s.misc = o; o = up(o + 512);     // the adapter set, abort flag, mbarriers
    s.total = o;
    return s;
}

struct Ctx {
    uint8_t* sm;
    LatSmem L;
    int warp, lane, g, t;
    uint32_t box_no;           // boxes that have gone through the weight ring so far (the same in every thread)
    uint32_t kv_no;            // head buffers filled so far
    int* status;
    volatile int* abort_flag;
};

__device__ __forceinline__ uint32_t ring_bar(const Ctx& cx, int slot) { return s_u32(cx.sm + cx.L.misc + 256) + 8u * slot; }
__device__ __forceinline__ uint32_t kv_bar(const Ctx& cx, int buf) { return s_u32(cx.sm + cx.L.misc + 256) + 8u * (LT_SLOTS + buf); }

// Bounded wait on a transaction barrier (every thread of the CTA may call it).  Once a wait has run out
// the CTA is aborting: later waits return at once and the results are meaningless (the status word says so).
__device__ __forceinline__ void bar_wait(const Ctx& cx, uint32_t bar, uint32_t parity) {
    if (bar_try(bar, parity)) return;
    const long long t0 = clock64();
    while (!bar_try(bar, parity)) {
        if (*cx.abort_flag) return;
        if (clock64() - t0 > LT_WAIT_CYCLES) {
            *cx.abort_flag = 1;
            atomicCAS(cx.status, 0, (int)PM_ERR_TIMEOUT);
            return;
        }
    }
}

struct LoraExp {               // LoRA expand of the current linear: t (shared memory) times B slabs (global)
    int n_act;
    int adapter[LT_MAX_SET], slabs[LT_MAX_SET];
    const bf16* Bt;
    int slabs_max, rs;         // rs: columns of t per adapter
};

// y[16, N] = A[16, K] W + LoRA expand, handed element-wise to epi(row, n, value).  A: bf16 in shared memory
// with row stride lda; rows [row0, row0 + N) of the [*, K] matrix behind `tm` come through the ring as TMA
// boxes of [box_rows outputs][64 inputs] (box_rows = 128 for the weights: two n8 tiles per warp; 16 for a
// LoRA slab of A^T: warp 0 alone).  All threads of the CTA call it; lane 0 of warps 0..2 issues the copies.
// col0 / col1: optional per-output-column vectors (bias; LayerNorm g or c1 ...); a thread's four values of
// each are fetched while the last K box is still being multiplied and handed to epi, so that the epilogue's
// stores never sit between a load and its use.
template <typename Epi>
__device__ void linear16(Ctx& cx, const bf16* A, int lda, const CUtensorMap* tm, int box_rows, int row0, int N, int K,
                         const LoraExp* lx, const float* col0, const float* col1, Epi epi) {
    const int n_chunks = (N + box_rows - 1) / box_rows, k_boxes = K >> 6;
    // boxes go through the ring in groups of up to LT_GROUP consecutive K boxes of one chunk of outputs: one
    // CTA-wide barrier per group, and while a group is multiplied the next one is on its way
    const int gpc = (k_boxes + LT_GROUP - 1) / LT_GROUP, n_groups = n_chunks * gpc;
    const uint32_t a_base = s_u32(A), ring = s_u32(cx.sm + cx.L.region), t_base = s_u32(cx.sm + cx.L.tbuf);
    const int lane = cx.lane, warp = cx.warp;
    uint32_t issued = cx.box_no;                      // number of the next box to issue (the same in every thread)
    auto issue_group = [&](int g) {
        const int nc = g / gpc, kb0 = (g % gpc) * LT_GROUP, nb = min(LT_GROUP, k_boxes - kb0);
        if (lane == 0 && warp < nb) {                 // box j of the group: lane 0 of warp j
            const int slot = (int)((issued + (uint32_t)warp) % LT_SLOTS);
            bar_expect(ring_bar(cx, slot), (uint32_t)box_rows * 128u);
            tma_box(ring + slot * LT_BOX_BYTES, tm, (kb0 + warp) * 64, row0 + nc * box_rows, ring_bar(cx, slot));
        }
        issued += (uint32_t)nb;
    };
    issue_group(0);
    float acc[2][4];
    const int row16 = warp * 16;                   // this warp's rows of a box
    const int mi = lane >> 3;
    const int r = row16 + (mi >> 1) * 8 + (lane & 7);
    for (int g = 0; g < n_groups; ++g) {
        // the slots freed by the previous group (everyone is past its closing barrier) take the next one
        if (g + 1 < n_groups) issue_group(g + 1);
        const int nc = g / gpc, kb0 = (g % gpc) * LT_GROUP, nb = min(LT_GROUP, k_boxes - kb0);
        const bool last = kb0 + nb == k_boxes;
        if (kb0 == 0) {
#pragma unroll
            for (int q = 0; q < 2; ++q) acc[q][0] = acc[q][1] = acc[q][2] = acc[q][3] = 0.f;
        }
        const int n16 = nc * box_rows + row16;
        const bool active = row16 < box_rows && n16 < N;
        float cv0[2][2] = {{0.f, 0.f}, {0.f, 0.f}}, cv1[2][2] = {{0.f, 0.f}, {0.f, 0.f}};
        if (active && last) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int n = n16 + q * 8 + 2 * cx.t;
                if (n16 + q * 8 < N) {
                    if (col0) { const float2 v = __ldg(reinterpret_cast<const float2*>(col0 + n)); cv0[q][0] = v.x; cv0[q][1] = v.y; }
                    if (col1) { const float2 v = __ldg(reinterpret_cast<const float2*>(col1 + n)); cv1[q][0] = v.x; cv1[q][1] = v.y; }
                }
            }
        }
        for (int j = 0; j < nb; ++j) {
            const uint32_t no = cx.box_no + (uint32_t)j;
            const int slot = (int)(no % LT_SLOTS);
            bar_wait(cx, ring_bar(cx, slot), (no / LT_SLOTS) & 1u);
            if (active) {
                const uint32_t a_row = a_base + ((lane & 15) * lda + (kb0 + j) * 64 + (lane >> 4) * 8) * 2;
                const uint32_t box = ring + slot * LT_BOX_BYTES;
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    uint32_t a[4], b0, b1, b2, b3;
                    ldsm4(a_row + ks * 32, a[0], a[1], a[2], a[3]);
                    const int c = ks * 2 + (mi & 1);
                    ldsm4(box + r * 128 + ((c ^ (r & 7)) << 4), b0, b1, b2, b3);
                    mma16816(acc[0], a, b0, b1);
                    mma16816(acc[1], a, b2, b3);
                }
            }
        }
        cx.box_no += (uint32_t)nb;
        if (active && last) {
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int n8 = n16 + q * 8;
                if (n8 >= N) break;
                if (lx) {
                    for (int p = 0; p < lx->n_act; ++p)
                        for (int sl = 0; sl < lx->slabs[p]; ++sl) {
                            uint32_t a[4];
                            ldsm4(t_base + ((lane & 15) * cx.L.ldt + p * lx->rs + sl * 16 + (lane >> 4) * 8) * 2, a[0], a[1], a[2], a[3]);
                            const bf16* bp = lx->Bt + (((size_t)(lx->adapter[p] * lx->slabs_max + sl) * N) + n8 + cx.g) * PM_SLAB;
                            const uint32_t b0 = __ldg(reinterpret_cast<const unsigned int*>(bp + 2 * cx.t));
                            const uint32_t b1 = __ldg(reinterpret_cast<const unsigned int*>(bp + 2 * cx.t + 8));
                            mma16816(acc[q], a, b0, b1);
                        }
                }
                const int n = n8 + 2 * cx.t;
                epi(cx.g, n, acc[q][0], cv0[q][0], cv1[q][0]); epi(cx.g, n + 1, acc[q][1], cv0[q][1], cv1[q][1]);
                epi(cx.g + 8, n, acc[q][2], cv0[q][0], cv1[q][0]); epi(cx.g + 8, n + 1, acc[q][3], cv0[q][1], cv1[q][1]);
            }
        }
        __syncthreads();          // the group's slots are refilled by the next iteration's copies
    }
}

__device__ __forceinline__ float gelu_exact(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752440f)); }

// abuf <- bf16(xres); stats[r] = (mean, rstd, 1/rstd) of the rounded row (what the tensor cores multiply)
__device__ void round_rows_and_stats(Ctx& cx, int d, float eps) {
    const float* x = reinterpret_cast<const float*>(cx.sm + cx.L.xres);
    bf16* a = reinterpret_cast<bf16*>(cx.sm + cx.L.abuf);
    float4* st = reinterpret_cast<float4*>(cx.sm + cx.L.stats);
    for (int r = cx.warp; r < LT_ROWS; r += LT_WARPS) {
        float v[12];                                        // d <= 384
        float sum = 0.f;
#pragma unroll
        for (int i = 0; i < 12; ++i) {
            const int c = cx.lane + 32 * i;
            v[i] = 0.f;
            if (c < d) {
                const bf16 h = __float2bfloat16_rn(x[r * d + c]);
                a[r * cx.L.lda + c] = h;
                v[i] = __bfloat162float(h);
                sum += v[i];
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        const float mean = sum / (float)d;
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < 12; ++i) if (cx.lane + 32 * i < d) { const float t = v[i] - mean; sq += t * t; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
        const float rstd = rsqrtf(sq / (float)d + eps);
        if (cx.lane == 0) st[r] = make_float4(mean, rstd, 1.f / rstd, 0.f);
    }
}

struct ActiveSet { int n; int id[LT_MAX_SET]; int slabs[LT_MAX_SET]; float scale[LT_MAX_SET]; };

// LoRA shrink for the adapters of `as` that touch `lin`: t[r][p * rs + j] (bf16) = s_a (x A_a) (folded
// linears: s_a ((x A' - mean c1) + c2 / rstd), the fused accumulator being scaled by rstd afterwards).
// Returns the expand description (adapters in ascending id).
__device__ void lora_shrink(Ctx& cx, const LatLinear& lin, const ActiveSet& as, int slabs_max, const bf16* A, int lda,
                            LoraExp* lx) {
    lx->n_act = 0; lx->Bt = lin.Bt; lx->slabs_max = slabs_max; lx->rs = slabs_max * PM_SLAB;
    if (!lin.At) return;
    const float4* st = reinterpret_cast<const float4*>(cx.sm + cx.L.stats);
    bf16* tb = reinterpret_cast<bf16*>(cx.sm + cx.L.tbuf);
    for (int i = 0; i < as.n; ++i) {
        const int a = as.id[i];
        if (!((lin.adapted[a >> 5] >> (a & 31)) & 1u)) continue;
        const int p = lx->n_act++;
        lx->adapter[p] = a; lx->slabs[p] = as.slabs[i];
        const int rs_a = as.slabs[i] * PM_SLAB;
        const float sc = as.scale[i];
        const float* c1 = lin.c1 ? lin.c1 + (size_t)a * lx->rs : nullptr;
        const float* c2 = lin.c2 ? lin.c2 + (size_t)a * lx->rs : nullptr;
        const bool folded = lin.ln_g != nullptr;
        const int ldt = cx.L.ldt, col0 = p * lx->rs;
        linear16(cx, A, lda, &lin.tm_at, PM_SLAB, a * lx->rs, rs_a, lin.k_in, nullptr, folded ? c1 : nullptr, folded ? c2 : nullptr,
                 [&](int r, int j, float v, float c1j, float c2j) {
                     if (folded) v = (v - st[r].x * c1j) + c2j * st[r].z;
                     tb[r * ldt + col0 + j] = __float2bfloat16_rn(v * sc);
                 });
    }
    __syncthreads();
}

__global__ void __launch_bounds__(LT_THREADS, 1) latency_forward_kernel(const __grid_constant__ LatArgs args) {
    extern __shared__ __align__(1024) uint8_t smem[];
    if (s_u32(smem) & 1023u) {                 // swizzled boxes need a 1024-byte aligned window
        if (threadIdx.x == 0) atomicCAS(args.status, 0, (int)PM_ERR_CUDA);
        return;
    }
    Ctx cx;
    cx.sm = smem;
    cx.L = lat_layout(args.d, args.mlp, args.patch_dim, args.slabs_max * PM_SLAB * args.max_set, args.tokens);
    cx.warp = threadIdx.x >> 5; cx.lane = threadIdx.x & 31; cx.g = cx.lane >> 2; cx.t = cx.lane & 3;
    const int f = blockIdx.x / args.tiles_pf, rt = blockIdx.x % args.tiles_pf;     // slot, row tile
    const int frame = args.perm ? args.perm[f] : f;                                  // input / output row
    const int T = args.tokens, d = args.d, r0 = rt * LT_ROWS;
    const int tpad = (T + 15) / 16 * 16;
    float* xres = reinterpret_cast<float*>(smem + cx.L.xres);
    bf16* abuf = reinterpret_cast<bf16*>(smem + cx.L.abuf);
    bf16* hbuf = reinterpret_cast<bf16*>(smem + cx.L.hbuf);
    bf16* qbuf = reinterpret_cast<bf16*>(smem + cx.L.qbuf);
    const float4* stats = reinterpret_cast<const float4*>(smem + cx.L.stats);
    ActiveSet* as = reinterpret_cast<ActiveSet*>(smem + cx.L.misc);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + cx.L.misc + 192);
    cx.box_no = 0; cx.kv_no = 0; cx.status = args.status; cx.abort_flag = abort_flag;
    if (threadIdx.x == 0) {
        for (int i = 0; i < LT_SLOTS + 2; ++i) bar_init(ring_bar(cx, i), 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }

    // ---- the frame's adapter set: valid, registered, distinct ids in ascending order
    if (threadIdx.x == 0) {
        *abort_flag = 0;
        as->n = 0;
        const int o0 = args.set_off[f], cnt = args.set_off[f + 1] - o0;
        bool bad = cnt < 0 || o0 < 0;
        for (int i = 0; i < cnt && !bad; ++i) {
            const int a = args.set_ids[o0 + i];
            if (a < 0 || a >= args.max_adapters || args.rank[a] <= 0) { atomicCAS(args.status, 0, (int)PM_ERR_ARG); continue; }
            int at = 0;
            bool dup = false;
            while (at < as->n && as->id[at] <= a) { dup |= as->id[at] == a; ++at; }
            if (dup) { atomicCAS(args.status, 0, (int)PM_ERR_ARG); continue; }
            if (as->n == args.max_set) {                    // keep the lowest max_set ids
                atomicCAS(args.status, 0, (int)PM_ERR_CAPACITY);
                if (at == as->n) continue;
                --as->n;
            }
            for (int j = as->n; j > at; --j) as->id[j] = as->id[j - 1];
            as->id[at] = a;
            ++as->n;
        }
        if (bad) atomicCAS(args.status, 0, (int)PM_ERR_ARG);
        for (int i = 0; i < as->n; ++i) {
            as->slabs[i] = (args.rank[as->id[i]] + PM_SLAB - 1) / PM_SLAB;
            as->scale[i] = args.scale[as->id[i]];
        }
    }
    // ---- patch gather: hbuf[r][c*P*P + py*P + px] = frame[c][gy*P + py][gx*P + px] of token r0 + r (token 0 = CLS)
    {
        const int P = 16, per_row = args.patch_dim / 8;
        const bf16* fr = args.frames + (size_t)frame * 3 * args.img * args.img;
        for (int i = threadIdx.x; i < LT_ROWS * per_row; i += LT_THREADS) {
            const int r = i / per_row, ch = i % per_row, tok = r0 + r;
            uint4 v = make_uint4(0, 0, 0, 0);
            if (tok >= 1 && tok < T) {
                const int p = tok - 1, gy = p / args.grid, gx = p % args.grid;
                const int col = ch * 8, c = col / (P * P), py = (col / P) % P, px = col % P;
                v = *reinterpret_cast<const uint4*>(fr + ((size_t)c * args.img + gy * P + py) * args.img + gx * P + px);
            }
            *reinterpret_cast<uint4*>(hbuf + r * cx.L.ldh + ch * 8) = v;
        }
    }
    __syncthreads();
    const ActiveSet aset = *as;
    // ---- patch projection + positions; the CLS row
    const LatLinear* patch = args.lin + (size_t)args.layers * 4;
    const float* patch_bias = patch->bias;
    linear16(cx, hbuf, cx.L.ldh, &patch->tm_w, 128, 0, d, args.patch_dim, nullptr, patch_bias, nullptr, [&](int r, int n, float v, float b, float) {
        const int tok = r0 + r;
        float out = 0.f;
        if (tok == 0) out = args.cls[n] + args.pos[n];
        else if (tok < T) out = v + b + args.pos[(size_t)tok * d + n];
        xres[r * d + n] = out;                              // rows past the frame stay zero
    });
    __syncthreads();

    LoraExp lx;
    const float att_scale = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) * log2(e)
    for (int l = 0; l < args.layers; ++l) {
        const LatLinear* lin = args.lin + (size_t)l * 4;
        bf16* kvb = args.kv + (size_t)(l & 1) * args.n_frames * T * 2 * d + (size_t)f * T * 2 * d;
        // ---- qkv (LayerNorm 1 folded): q stays here, k and v go to the frame's exchange buffer
        round_rows_and_stats(cx, d, args.eps);
        __syncthreads();
        lora_shrink(cx, lin[0], aset, args.slabs_max, abuf, cx.L.lda, &lx);
        {
            const float* lg = lin[0].ln_g; const float* bb = lin[0].bias;
            linear16(cx, abuf, cx.L.lda, &lin[0].tm_w, 128, 0, 3 * d, d, lx.n_act ? &lx : nullptr, bb, lg, [&](int r, int n, float v, float b, float gsum) {
                const float y = stats[r].y * (v - stats[r].x * gsum) + b;
                if (n < d) qbuf[r * cx.L.ldq + n] = __float2bfloat16_rn(y);
                else if (r0 + r < T) kvb[(size_t)(r0 + r) * 2 * d + (n - d)] = __float2bfloat16_rn(y);
            });
        }
        // ---- the CTAs of the frame meet: all keys and values of this block are in place (they were written
        // with ordinary stores and are fetched by TMA on the other side: order the two proxies as well)
        asm volatile("fence.proxy.async.global;" ::: "memory");
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0 && !*abort_flag) {
            atomicAdd(args.bar + f, 1u);
            const unsigned int want = (unsigned int)args.tiles_pf * (unsigned int)(l + 1);
            const long long t0 = clock64();
            unsigned int seen;
            do {
                asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(args.bar + f) : "memory");
                if (seen < want && clock64() - t0 > LT_WAIT_CYCLES) {
                    *abort_flag = 1;
                    atomicCAS(args.status, 0, (int)PM_ERR_TIMEOUT);
                    break;
                }
            } while (seen < want);
        }
        __syncthreads();
        if (*abort_flag) break;
        // ---- attention, head by head: the warps split the keys, then merge their partial results
        // keys and values of a head arrive as two TMA boxes ([tpad rows][64 dims], 128B swizzle; rows past
        // the frame hold a neighbour's rows or zeros and are masked below); the next head's are on their
        // way while this one is computed
        const int kv_row0 = ((l & 1) * args.n_frames + f) * T;
        auto fetch_head = [&](int h) {
            const int buf = (int)(cx.kv_no & 1u);
            const uint32_t dst = s_u32(smem + cx.L.region) + buf * cx.L.kv_head;
            bar_expect(kv_bar(cx, buf), 2u * (uint32_t)tpad * 128u);
            tma_box(dst, &args.tm_kv, h * LT_HD, kv_row0, kv_bar(cx, buf));
            tma_box(dst + cx.L.kv_head / 2, &args.tm_kv, d + h * LT_HD, kv_row0, kv_bar(cx, buf));
        };
        if (threadIdx.x == 0) {
            asm volatile("fence.proxy.async.global;" ::: "memory");
            fetch_head(0);
        }
        for (int h = 0; h < args.heads; ++h) {
            const int buf = (int)(cx.kv_no & 1u);
            uint8_t* Ks = smem + cx.L.region + buf * cx.L.kv_head;
            uint8_t* Vs = Ks + cx.L.kv_head / 2;
            bar_wait(cx, kv_bar(cx, buf), (cx.kv_no >> 1) & 1u);
            ++cx.kv_no;
            // the other buffer was last read by head h - 1, and everyone is past that head's closing barrier
            if (threadIdx.x == 0 && h + 1 < args.heads) fetch_head(h + 1);
            const int n_t8 = tpad / 8;
            const int t8_lo = (n_t8 * cx.warp) / LT_WARPS, t8_hi = (n_t8 * (cx.warp + 1)) / LT_WARPS;    // at most 4 tiles
            const uint32_t ks_addr = s_u32(Ks), vs_addr = s_u32(Vs);
            float s[4][4];
            uint32_t qa[4][4];
#pragma unroll
            for (int ks = 0; ks < 4; ++ks)
                ldsm4(s_u32(qbuf) + ((cx.lane & 15) * cx.L.ldq + h * LT_HD + ks * 16 + (cx.lane >> 4) * 8) * 2,
                      qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
            float m_lo = -INFINITY, m_hi = -INFINITY;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
                const int t8 = t8_lo + j;
                if (t8 < t8_hi) {
#pragma unroll
                    for (int ks = 0; ks < 4; ++ks) {
                        const int r = t8 * 8 + (cx.lane & 7), c = ks * 2 + ((cx.lane >> 3) & 1);
                        uint32_t b0, b1;
                        ldsm2(ks_addr + r * 128 + ((c ^ (r & 7)) << 4), b0, b1);
                        mma16816(s[j], qa[ks], b0, b1);
                    }
                }
                const int key = t8 * 8 + 2 * cx.t;
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                    const bool ok = t8 < t8_hi && key + (e & 1) < T;
                    s[j][e] = ok ? s[j][e] * att_scale : -INFINITY;
                }
                m_lo = fmaxf(m_lo, fmaxf(s[j][0], s[j][1]));
                m_hi = fmaxf(m_hi, fmaxf(s[j][2], s[j][3]));
            }
            m_lo = fmaxf(m_lo, __shfl_xor_sync(0xFFFFFFFFu, m_lo, 1));
            m_lo = fmaxf(m_lo, __shfl_xor_sync(0xFFFFFFFFu, m_lo, 2));
            m_hi = fmaxf(m_hi, __shfl_xor_sync(0xFFFFFFFFu, m_hi, 1));
            m_hi = fmaxf(m_hi, __shfl_xor_sync(0xFFFFFFFFu, m_hi, 2));
            // a warp whose keys are all beyond the frame contributes nothing (its maximum stays -inf)
            const float ms_lo = m_lo == -INFINITY ? 0.f : m_lo, ms_hi = m_hi == -INFINITY ? 0.f : m_hi;
            float l_lo = 0.f, l_hi = 0.f;
            uint32_t pa[2][4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float p0 = exp2f(s[j][0] - ms_lo), p1 = exp2f(s[j][1] - ms_lo);
                const float p2 = exp2f(s[j][2] - ms_hi), p3 = exp2f(s[j][3] - ms_hi);
                l_lo += p0 + p1;
                l_hi += p2 + p3;
                pa[j >> 1][(j & 1) * 2 + 0] = pk_bf16(p0, p1);
                pa[j >> 1][(j & 1) * 2 + 1] = pk_bf16(p2, p3);
            }
            l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 1);
            l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 2);
            l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 1);
            l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 2);
            float o[8][4];
#pragma unroll
            for (int i = 0; i < 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
#pragma unroll
            for (int kk = 0; kk < 2; ++kk) {                 // 16-key steps of this warp's keys
                if (t8_lo + 2 * kk < t8_hi) {
#pragma unroll
                    for (int n = 0; n < 4; ++n) {            // pairs of 8-dim tiles
                        const int mi = cx.lane >> 3;
                        // rows past the warp's range belong to a neighbour's keys: their probabilities are 0
                        const int r = min((t8_lo + 2 * kk) * 8 + (mi & 1) * 8 + (cx.lane & 7), tpad - 1);
                        const int c = n * 2 + (mi >> 1);
                        uint32_t b0, b1, b2, b3;
                        ldsm4t(vs_addr + r * 128 + ((c ^ (r & 7)) << 4), b0, b1, b2, b3);
                        mma16816(o[2 * n], pa[kk], b0, b1);
                        mma16816(o[2 * n + 1], pa[kk], b2, b3);
                    }
                }
            }
            // partial results: part[warp][row][0..63] = o, [64] = max, [65] = sum
            float* part = reinterpret_cast<float*>(smem + cx.L.part) + (size_t)cx.warp * LT_ROWS * (LT_HD + 2);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                const int c = i * 8 + 2 * cx.t;
                part[cx.g * (LT_HD + 2) + c] = o[i][0]; part[cx.g * (LT_HD + 2) + c + 1] = o[i][1];
                part[(cx.g + 8) * (LT_HD + 2) + c] = o[i][2]; part[(cx.g + 8) * (LT_HD + 2) + c + 1] = o[i][3];
            }
            if (cx.t == 0) {
                part[cx.g * (LT_HD + 2) + 64] = m_lo; part[cx.g * (LT_HD + 2) + 65] = l_lo;
                part[(cx.g + 8) * (LT_HD + 2) + 64] = m_hi; part[(cx.g + 8) * (LT_HD + 2) + 65] = l_hi;
            }
            __syncthreads();
            {   // merge: thread -> (row, four dims)
                const float* pall = reinterpret_cast<const float*>(smem + cx.L.part);
                const int r = threadIdx.x >> 4, c4 = (threadIdx.x & 15) * 4;
                float m = -INFINITY;
#pragma unroll
                for (int w = 0; w < LT_WARPS; ++w) m = fmaxf(m, pall[(w * LT_ROWS + r) * (LT_HD + 2) + 64]);
                float den = 0.f, num[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int w = 0; w < LT_WARPS; ++w) {
                    const float* pr = pall + (w * LT_ROWS + r) * (LT_HD + 2);
                    const float e = pr[64] == -INFINITY ? 0.f : exp2f(pr[64] - m);
                    den += e * pr[65];
#pragma unroll
                    for (int q = 0; q < 4; ++q) num[q] += e * pr[c4 + q];
                }
                const float inv = 1.f / den;                 // key 0 is always valid: den > 0
                uint2 pkd;
                pkd.x = pk_bf16(num[0] * inv, num[1] * inv);
                pkd.y = pk_bf16(num[2] * inv, num[3] * inv);
                *reinterpret_cast<uint2*>(abuf + r * cx.L.lda + h * LT_HD + c4) = pkd;
            }
            __syncthreads();
        }
        // ---- proj (+ residual)
        lora_shrink(cx, lin[1], aset, args.slabs_max, abuf, cx.L.lda, &lx);
        {
            const float* bb = lin[1].bias;
            linear16(cx, abuf, cx.L.lda, &lin[1].tm_w, 128, 0, d, d, lx.n_act ? &lx : nullptr, bb, nullptr,
                     [&](int r, int n, float v, float b, float) { if (r0 + r < T) xres[r * d + n] += v + b; });
        }
        __syncthreads();
        // ---- fc1 (LayerNorm 2 folded, GELU) and fc2 (+ residual)
        round_rows_and_stats(cx, d, args.eps);
        __syncthreads();
        lora_shrink(cx, lin[2], aset, args.slabs_max, abuf, cx.L.lda, &lx);
        {
            const float* lg = lin[2].ln_g; const float* bb = lin[2].bias;
            linear16(cx, abuf, cx.L.lda, &lin[2].tm_w, 128, 0, args.mlp, d, lx.n_act ? &lx : nullptr, bb, lg, [&](int r, int n, float v, float b, float gsum) {
                hbuf[r * cx.L.ldh + n] = __float2bfloat16_rn(gelu_exact(stats[r].y * (v - stats[r].x * gsum) + b));
            });
        }
        __syncthreads();
        lora_shrink(cx, lin[3], aset, args.slabs_max, hbuf, cx.L.ldh, &lx);
        {
            const float* bb = lin[3].bias;
            linear16(cx, hbuf, cx.L.ldh, &lin[3].tm_w, 128, 0, d, args.mlp, lx.n_act ? &lx : nullptr, bb, nullptr,
                     [&](int r, int n, float v, float b, float) { if (r0 + r < T) xres[r * d + n] += v + b; });
        }
        __syncthreads();
    }

    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // copies still in flight land before shared memory goes away
        return;
    }
    if (rt != 0) return;

    // ---- heads on the CLS row (row 0 of the frame's first CTA): final LayerNorm, base head, adapter heads
    float* z = reinterpret_cast<float*>(smem + cx.L.region);
    if (cx.warp == 0) {
        float v[12], sum = 0.f;
#pragma unroll
        for (int i = 0; i < 12; ++i) { const int c = cx.lane + 32 * i; v[i] = c < d ? xres[c] : 0.f; sum += v[i]; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xFFFFFFFFu, sum, o);
        const float mean = sum / (float)d;
        float sq = 0.f;
#pragma unroll
        for (int i = 0; i < 12; ++i) if (cx.lane + 32 * i < d) { const float t = v[i] - mean; sq += t * t; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) sq += __shfl_xor_sync(0xFFFFFFFFu, sq, o);
        const float rstd = rsqrtf(sq / (float)d + args.eps);
#pragma unroll
        for (int i = 0; i < 12; ++i) {
            const int c = cx.lane + 32 * i;
            if (c < d) z[c] = (v[i] - mean) * rstd * args.lnf_g[c] + args.lnf_b[c];
        }
    }
    float* srow = args.scores_out + (size_t)frame * args.n_classes;
    for (int k = threadIdx.x; k < args.n_classes; k += LT_THREADS) srow[k] = 0.f;
    __syncthreads();
    auto dot = [&](const bf16* w) {
        float acc = 0.f;
        for (int c = cx.lane * 2; c < d; c += 64) {
            const __nv_bfloat162 h2 = *reinterpret_cast<const __nv_bfloat162*>(w + c);
            acc = fmaf(z[c], __bfloat162float(h2.x), fmaf(z[c + 1], __bfloat162float(h2.y), acc));
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, o);
        return acc;
    };
    if (args.base_out) {
        for (int k = cx.warp; k < args.n_classes; k += LT_WARPS) {
            const float v = dot(args.head_wt + (size_t)k * d) + args.head_b[k];
            if (cx.lane == 0) args.base_out[(size_t)frame * args.n_classes + k] = 1.f / (1.f + expf(-v));
        }
    }
    for (int i = 0; i < aset.n; ++i) {
        const int a = aset.id[i];
        for (int r = args.hoff[a] + cx.warp; r < args.hoff[a + 1]; r += LT_WARPS) {
            const float v = dot(args.hcat + (size_t)r * d) + args.hbias[r];
            // scores are positive: the maximum over adapters is an integer maximum of the bit patterns
            if (cx.lane == 0) atomicMax(reinterpret_cast<int*>(srow + args.hcls[r]), __float_as_int(1.f / (1.f + expf(-v))));
        }
    }
}

}  // namespace

size_t latency_smem_bytes(int d, int mlp, int patch_dim, int rs_total, int tokens) {
    return (size_t)lat_layout(d, mlp, patch_dim, rs_total, tokens).total;
}

cudaError_t launch_latency_forward(const Launch& L, const LatArgs& a) {
    const size_t smem = latency_smem_bytes(a.d, a.mlp, a.patch_dim, a.slabs_max * PM_SLAB * a.max_set, a.tokens);
    static SmemGrant grant;
    if (cudaError_t e = grant.ensure(latency_forward_kernel, (int)smem); e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(a.n_frames * a.tiles_pf);
    cfg.blockDim = dim3(LT_THREADS);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = L.st;
    // the CTAs of a frame wait for one another: all of them must be resident at once
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    ProfScope ps(L, KC_GEMM);
    LatArgs copy = a;
    copy.status = L.status;
    // the frames' arrival counters start at zero (an aborted launch may have left them anywhere)
    cudaError_t e = cudaMemsetAsync(a.bar, 0, sizeof(unsigned int) * a.n_frames, L.st);
    if (e != cudaSuccess) return e;
    e = cudaLaunchKernelEx(&cfg, latency_forward_kernel, copy);
    BUMP(L);
    return e != cudaSuccess ? e : cudaGetLastError();
}
