// Whole-network kernel for a handful of frames (the single-stream operating point of Sec. 4): patch
// embedding, all encoder blocks with their unmerged LoRA terms (Sec. 3.1), final LayerNorm, base and
// adapter heads with sigmoid and merge (Fig. 5b) in ONE launch.
//
// Everything in a ViT block except attention is local to a token row, so a CTA owns 16 token rows of one
// frame from the first layer to the last and keeps their residual stream (fp32) and every intermediate in
// shared memory.  What a CTA reads from L2 is static -- weights, LoRA slabs, bias vectors, in an order that
// is known when the kernel starts -- so one producer thread walks that order and keeps a ring of 32 KB
// shared-memory slots full by TMA, across the boundaries of linears and blocks, while the eight consumer
// warps multiply what has landed (full / empty transaction barriers per slot, no CTA-wide barrier in the
// stream).  Every CTA reads every weight, 13 CTAs per frame.
// The one exchange per block is attention: each CTA publishes the keys and values of its rows (two global
// buffers used in turn) as soon as those columns of the qkv product are done, counts itself in at the
// frame's counter and goes on with the query columns; a second producer thread waits for the counter
// (bounded) and fetches the heads' keys and values, the next head's while this one is computed.  Each CTA
// attends from its 16 query rows to all keys of its frame: four warp pairs split the keys, the two warps
// of a pair split the head dimension, partial softmax results are merged through shared memory.
// Contractions run on mma.sync m16n8k16 (bf16 in, fp32 accumulate): with 16 rows per CTA there is no
// 128-row tile to give to tcgen05.
// LayerNorm uses the folded form the other kernels use: y = rstd (x W' - mean g) + b'.
#include "common.cuh"

#define BUMP(L) do { if ((L).launches) ++*(L).launches; } while (0)

namespace {

constexpr int LT_ROWS = 16;
constexpr int LT_CWARPS = 8;                 // consumer warps
constexpr int LT_CTHREADS = LT_CWARPS * 32;
constexpr int LT_THREADS = LT_CTHREADS + 64; // + the weight producer's warp + the key/value producer's warp
constexpr int LT_BOX_BYTES = 128 * 128;      // [128 output rows][64 bf16 inputs], 128B swizzle
constexpr int LT_SLOT_BYTES = 2 * LT_BOX_BYTES;  // a ring step: two K boxes of a chunk of outputs
constexpr int LT_MAX_SLOTS = 8;
constexpr int LT_MAX_SET = 8;
constexpr int LT_MAX_SLABS = 8;              // active LoRA slabs of one linear
constexpr int LT_HD = 64;
constexpr int LT_KSPLIT = 4;                 // key ranges of the attention warps
constexpr int LT_ST = 8;                     // key tiles (8 keys) of one range, at most (256 tokens)
constexpr long long LT_WAIT_CYCLES = 4000000000ll;

__device__ __forceinline__ uint32_t s_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void ldsm4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
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
__device__ __forceinline__ float ex2(float x) {            // 2^x, one special-function instruction; 2^-inf = 0
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
__device__ __forceinline__ uint32_t pk_bf16(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ void bar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_expect(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
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

// untiled copy: both addresses 16-byte aligned, bytes a multiple of 16
__device__ __forceinline__ void bulk_copy(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void consumer_sync() { asm volatile("bar.sync 1, %0;" ::"n"(LT_CTHREADS) : "memory"); }

}  // namespace

namespace {

struct LatSmem {               // offsets (bytes) into dynamic shared memory
    int ring, kbuf, vbuf, xres, abuf, qbuf, hbuf, tbuf, stats, colv, slabs, misc, total;
    int lda, ldh, ldq, ldt;    // row strides in bf16 elements
    int kv_bytes;              // one head's keys (or values): [tpad rows][128 bytes], and a kilobyte behind them
    int cv_floats;             // one vector pack: bias[nmax], g[nmax], c1[128], c2[128]
};

__host__ __device__ inline LatSmem lat_layout(int d, int mlp, int patch_dim, int tokens, int layers, int slots) {
    LatSmem s;
    auto up = [](int v) { return (v + 127) & ~127; };
    const int wide = mlp > patch_dim ? mlp : patch_dim, nmax = 3 * d > mlp ? 3 * d : mlp;
    s.lda = d + 8; s.ldh = wide + 8; s.ldq = d + 8; s.ldt = LT_MAX_SLABS * PM_SLAB + 8;
    const int tpad = (tokens + 15) / 16 * 16;
    s.kv_bytes = ((tpad * 128 + 1023) & ~1023) + 1024;      // + 1 KB that stays zero behind the values (see the P V loop)
    s.cv_floats = 2 * nmax + 2 * LT_MAX_SLABS * PM_SLAB;
    int o = 0;
    s.ring = o; o += slots * LT_SLOT_BYTES;                      // 1024-byte aligned, as the 128B swizzle wants
    s.kbuf = o; o += s.kv_bytes;
    s.vbuf = o; o += s.kv_bytes;
    s.xres = o; o = up(o + LT_ROWS * d * 4);
    s.abuf = o; o = up(o + LT_ROWS * s.lda * 2);
    s.qbuf = o; o = up(o + LT_ROWS * s.ldq * 2);
    // the MLP's hidden rows (and the gathered patches); between blocks' MLPs: the attention warps' partial results
    const int hb = LT_ROWS * s.ldh * 2, pb = LT_KSPLIT * LT_ROWS * (LT_HD + 2) * 4;
    s.hbuf = o; o = up(o + (hb > pb ? hb : pb));
    s.tbuf = o; o = up(o + LT_ROWS * s.ldt * 2);
    s.stats = o; o = up(o + LT_ROWS * 16);
    s.colv = o; o = up(o + 2 * s.cv_floats * 4);
    s.slabs = o; o = up(o + layers * 4 * 32);
    s.misc = o; o = up(o + 512);     // the adapter set, abort flag, mbarriers
    s.total = o;
    return s;
}

struct ActiveSet { int n; int id[LT_MAX_SET]; int slabs[LT_MAX_SET]; float scale[LT_MAX_SET]; };
// the LoRA slabs one linear applies to this frame: slab i belongs to set member who[i] and is its slab sl[i]
struct SlabTab { int n; uint8_t who[LT_MAX_SLABS]; uint8_t sl[LT_MAX_SLABS]; int pad[3]; };
static_assert(sizeof(SlabTab) == 32, "one table entry is 32 bytes");
static_assert(sizeof(ActiveSet) <= 128, "the adapter set sits in the first 128 bytes of the last region");

struct Ctx {
    uint8_t* sm;
    LatSmem L;
    int warp, lane, g, t, ns;
    uint32_t slot, phase;      // ring position: the same in every consumer thread (and in the producer)
    uint32_t li;               // linears done so far (their vector packs alternate between two buffers)
    int* status;
    volatile int* abort_flag;
};

__device__ __forceinline__ uint32_t bars(const Ctx& cx) { return s_u32(cx.sm + cx.L.misc + 256); }
__device__ __forceinline__ uint32_t full_bar(const Ctx& cx, uint32_t i) { return bars(cx) + 8u * i; }
__device__ __forceinline__ uint32_t empty_bar(const Ctx& cx, uint32_t i) { return bars(cx) + 64u + 8u * i; }
__device__ __forceinline__ uint32_t kfull_bar(const Ctx& cx) { return bars(cx) + 128u; }
__device__ __forceinline__ uint32_t kempty_bar(const Ctx& cx) { return bars(cx) + 136u; }
__device__ __forceinline__ uint32_t vfull_bar(const Ctx& cx) { return bars(cx) + 144u; }
__device__ __forceinline__ uint32_t vempty_bar(const Ctx& cx) { return bars(cx) + 152u; }
__device__ __forceinline__ uint32_t cfull_bar(const Ctx& cx, uint32_t b) { return bars(cx) + 160u + 8u * b; }
__device__ __forceinline__ uint32_t cempty_bar(const Ctx& cx, uint32_t b) { return bars(cx) + 176u + 8u * b; }
__device__ __forceinline__ uint32_t kvdone_bar(const Ctx& cx, uint32_t part) { return bars(cx) + 192u + 8u * part; }

// The order in which a linear's chunks of 128 outputs are taken (producer and consumers alike).  qkv (width d):
// the chunk with the first head's keys, the chunk with its values, the other chunks with key or value
// columns, then the chunks of query columns alone -- the frame's other CTAs can fetch the first head's keys
// and values, and then the others', while this CTA is still multiplying.  Every other linear: as they come.
struct ChunkOrder { int n_chunks, ck, cv, n_kv; bool qkv, reorder; };
__device__ __forceinline__ ChunkOrder chunk_order(int N, int d, bool qkv) {
    ChunkOrder o;
    o.n_chunks = (N + 127) >> 7; o.qkv = qkv; o.reorder = qkv && o.n_chunks > 2;
    o.ck = d >> 7; o.cv = (2 * d) >> 7; o.n_kv = o.n_chunks - o.ck;
    return o;
}
__device__ __forceinline__ int chunk_at(const ChunkOrder& o, int i) {
    if (!o.reorder) return i;
    if (i == 0) return o.ck;
    if (i == 1) return o.cv;
    const int j = i - 2, rest = o.n_kv - 2;              // chunks with key / value columns besides ck and cv
    if (j >= rest) return j - rest;                      // query columns alone: chunks 0 .. ck - 1
    const int c = o.ck + 1 + j;
    return c >= o.cv ? c + 1 : c;
}
// position after which the first head's (part 0) / all heads' (part 1) keys and values of this CTA are stored;
// a qkv of one or two chunks is not reordered and reports once, at its end
__device__ __forceinline__ int publish_pos(const ChunkOrder& o, int part) {
    if (!o.qkv) return -1;
    if (!o.reorder) return part == 0 ? -1 : o.n_chunks - 1;
    return part == 0 ? 1 : o.n_kv - 1;
}

// Bounded wait on a barrier.  Once a wait has run out the CTA is aborting: later waits return at once and
// the results are meaningless (the status word says so).
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
__device__ __forceinline__ void ring_advance(Ctx& cx) {
    if (++cx.slot == (uint32_t)cx.ns) { cx.slot = 0; cx.phase ^= 1u; }
}
// consumer side of one ring step: wait until the slot's copies have landed / hand the slot back
__device__ __forceinline__ uint32_t step_acquire(Ctx& cx) {
    bar_wait(cx, full_bar(cx, cx.slot), cx.phase);
    return s_u32(cx.sm + cx.L.ring) + cx.slot * LT_SLOT_BYTES;
}
__device__ __forceinline__ void step_release(Ctx& cx) {
    __syncwarp();
    if (cx.lane == 0) bar_arrive(empty_bar(cx, cx.slot));
    ring_advance(cx);
}
// producer side: wait until the eight consumer warps have handed the slot back (first lap: at once)
__device__ __forceinline__ uint32_t step_claim(Ctx& cx, uint32_t bytes) {
    bar_wait(cx, empty_bar(cx, cx.slot), cx.phase ^ 1u);
    bar_expect(full_bar(cx, cx.slot), bytes);
    return s_u32(cx.sm + cx.L.ring) + cx.slot * LT_SLOT_BYTES;
}

// What the weight producer sends for one linear, in this order (the consumers take it in the same order):
//   the vector pack (bias, g, c1, c2) into the linear's pack buffer;
//   LoRA shrink, if any slab is active: K/128 steps, each the [16 rows][64] boxes of A^T of all active slabs
//   for two K boxes (the second K box's slabs 16 KB into the slot);
//   for each chunk of 128 outputs, in the order of chunk_at(): K/128 steps of W^T, each two
//   K boxes of the chunk ([64 rows][64] boxes, two per K box of a full chunk), then the chunk's rows of
//   the active slabs' B^T ([128 rows][16] boxes, four per step).
__device__ void produce_linear(Ctx& cx, const LatLinear* lin, const SlabTab& st, const ActiveSet& as, int rs, int slabs_max,
                               int d, bool qkv) {
    const int N = lin->n_out, K = lin->k_in, k_boxes = K >> 6, n_chunks = (N + 127) >> 7, n_sl = st.n;
    const bool folded = lin->ln_g != nullptr;
    {
        const uint32_t b = cx.li & 1u, use = cx.li >> 1;
        bar_wait(cx, cempty_bar(cx, b), (use & 1u) ^ 1u);
        const uint32_t dst = s_u32(cx.sm + cx.L.colv) + b * (uint32_t)cx.L.cv_floats * 4u;
        const uint32_t vb = (uint32_t)N * 4u;
        const uint32_t bytes = vb + (folded ? vb : 0u) + (folded ? (uint32_t)n_sl * 128u : 0u);
        bar_expect(cfull_bar(cx, b), bytes);
        bulk_copy(dst, lin->bias, vb, cfull_bar(cx, b));
        if (folded) {
            bulk_copy(dst + vb, lin->ln_g, vb, cfull_bar(cx, b));
            for (int i = 0; i < n_sl; ++i) {
                const int arow = as.id[st.who[i]] * rs + st.sl[i] * PM_SLAB;
                bulk_copy(dst + 2u * vb + i * 64u, lin->c1 + arow, 64u, cfull_bar(cx, b));
                bulk_copy(dst + 2u * vb + LT_MAX_SLABS * 64u + i * 64u, lin->c2 + arow, 64u, cfull_bar(cx, b));
            }
        }
        ++cx.li;
    }
    if (n_sl) {
        for (int kb0 = 0; kb0 < k_boxes && !*cx.abort_flag; kb0 += 2) {
            const int nb = min(2, k_boxes - kb0);
            const uint32_t dst = step_claim(cx, (uint32_t)(nb * n_sl) * 2048u);
            for (int b = 0; b < nb; ++b)
                for (int i = 0; i < n_sl; ++i)
                    tma_box(dst + b * LT_BOX_BYTES + i * 2048u, &lin->tm_at, (kb0 + b) * 64, as.id[st.who[i]] * rs + st.sl[i] * PM_SLAB,
                            full_bar(cx, cx.slot));
            ring_advance(cx);
        }
    }
    const ChunkOrder order = chunk_order(N, d, qkv);
    for (int ci = 0; ci < n_chunks; ++ci) {
        const int nc = chunk_at(order, ci);
        const int rows = min(128, N - nc * 128);
        for (int kb0 = 0; kb0 < k_boxes && !*cx.abort_flag; kb0 += 2) {
            const int nb = min(2, k_boxes - kb0);
            const uint32_t dst = step_claim(cx, (uint32_t)(nb * rows) * 128u);
            for (int b = 0; b < nb; ++b)
                for (int hf = 0; hf * 64 < rows; ++hf)
                    tma_box(dst + b * LT_BOX_BYTES + hf * 8192u, &lin->tm_w, (kb0 + b) * 64, nc * 128 + hf * 64, full_bar(cx, cx.slot));
            ring_advance(cx);
        }
        for (int s0 = 0; s0 < n_sl && !*cx.abort_flag; s0 += 4) {
            const int cnt = min(4, n_sl - s0);
            const uint32_t dst = step_claim(cx, (uint32_t)cnt * 4096u);
            for (int j = 0; j < cnt; ++j) {
                const int i = s0 + j;
                tma_box(dst + j * 4096u, &lin->tm_bt, 0, (as.id[st.who[i]] * slabs_max + st.sl[i]) * N + nc * 128, full_bar(cx, cx.slot));
            }
            ring_advance(cx);
        }
    }
}

// one ring step of weights ([rows][64 inputs], this warp's 16 rows) against 64 columns of A (bf16, shared memory)
__device__ __forceinline__ void mma_step(Ctx& cx, uint32_t a_row0, int nb, bool active, float (&acc)[2][2][4]) {
    const uint32_t box0 = step_acquire(cx);
    if (active) {
        const int mi = cx.lane >> 3;
        const int r = cx.warp * 16 + (mi >> 1) * 8 + (cx.lane & 7);
        for (int bx = 0; bx < nb; ++bx) {
        const uint32_t box = box0 + bx * LT_BOX_BYTES, a_row = a_row0 + bx * 128;
        // all eight fetches first, then the eight multiplications (four independent accumulators in turn)
        uint32_t a[4][4], b[4][4];
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            ldsm4(a_row + ks * 32, a[ks][0], a[ks][1], a[ks][2], a[ks][3]);
            const int c = ks * 2 + (mi & 1);
            ldsm4(box + r * 128 + ((c ^ (r & 7)) << 4), b[ks][0], b[ks][1], b[ks][2], b[ks][3]);
        }
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            mma16816(acc[0][ks & 1], a[ks], b[ks][0], b[ks][1]);
            mma16816(acc[1][ks & 1], a[ks], b[ks][2], b[ks][3]);
        }
        }
    }
    step_release(cx);
}
__device__ __forceinline__ void acc_zero(float (&acc)[2][2][4]) {
#pragma unroll
    for (int q = 0; q < 2; ++q)
#pragma unroll
        for (int h = 0; h < 2; ++h) acc[q][h][0] = acc[q][h][1] = acc[q][h][2] = acc[q][h][3] = 0.f;
}

// The consumers' side of a linear's chunks: y[16, N] = A[16, K] W + t B.  A thread's eight values of a chunk
// go to epi(n0, y) in one call -- y[q][0..1] = columns n0 + 8 q, n0 + 8 q + 1 of row g, y[q][2..3] the same
// columns of row g + 8 -- so that the epilogue can fetch everything it needs before its first store.
// qkv: after the chunks at the two publish positions each warp reports at the barrier on which the key/value
// producer waits before it counts the CTA in at the frame's counter.
template <typename Epi>
__device__ void linear16(Ctx& cx, const bf16* A, int lda, int K, int N, int n_sl, int d, bool qkv,
                         Epi epi) {
    const int k_boxes = K >> 6, n_chunks = (N + 127) >> 7;
    const uint32_t a_base = s_u32(A) + ((cx.lane & 15) * lda + (cx.lane >> 4) * 8) * 2;
    const uint32_t t_row = s_u32(cx.sm + cx.L.tbuf) + ((cx.lane & 15) * cx.L.ldt + (cx.lane >> 4) * 8) * 2;
    const ChunkOrder order = chunk_order(N, d, qkv);
    for (int ci = 0; ci < n_chunks; ++ci) {
        const int nc = chunk_at(order, ci);
        const int rows = min(128, N - nc * 128);
        const bool active = cx.warp * 16 < rows;
        float acc[2][2][4];
        acc_zero(acc);
        for (int kb0 = 0; kb0 < k_boxes; kb0 += 2) mma_step(cx, a_base + kb0 * 128, min(2, k_boxes - kb0), active, acc);
        for (int s0 = 0; s0 < n_sl; s0 += 4) {
            const uint32_t box = step_acquire(cx);
            if (active) {
                // B^T rows are 32 bytes (16 ranks), 32B swizzle: the 16-byte half c of row n sits at c ^ ((n >> 2) & 1)
                const int n = cx.warp * 16 + ((cx.lane >> 4) & 1) * 8 + (cx.lane & 7), c = (cx.lane >> 3) & 1;
                const uint32_t b_row = box + n * 32 + ((c ^ ((n >> 2) & 1)) << 4);
                const int cnt = min(4, n_sl - s0);
                for (int j = 0; j < cnt; ++j) {
                    uint32_t a[4], b0, b1, b2, b3;
                    ldsm4(t_row + (s0 + j) * 32, a[0], a[1], a[2], a[3]);
                    ldsm4(b_row + j * 4096, b0, b1, b2, b3);
                    mma16816(acc[0][j & 1], a, b0, b1);
                    mma16816(acc[1][j & 1], a, b2, b3);
                }
            }
            step_release(cx);
        }
        if (active) {
            float y[2][4];
#pragma unroll
            for (int q = 0; q < 2; ++q)
#pragma unroll
                for (int e = 0; e < 4; ++e) y[q][e] = acc[q][0][e] + acc[q][1][e];
            epi(nc * 128 + cx.warp * 16 + 2 * cx.t, y);
        }
        // this warp's keys and values of the block (the first head's / all) are stored: tell the key/value producer
        if (ci == publish_pos(order, 0) || ci == publish_pos(order, 1)) {
            __syncwarp();
            if (cx.lane == 0) {
                if (ci == publish_pos(order, 0)) bar_arrive(kvdone_bar(cx, 0));
                if (ci == publish_pos(order, 1)) bar_arrive(kvdone_bar(cx, 1));
            }
        }
    }
}

// The consumers' side of a linear's shrink steps: warp i < n_sl multiplies the rows by slab i of A^T and
// hands epi(row, i, j, v[j], v[j + 1]) its 16 x 16 result (even j).
template <typename Epi>
__device__ void shrink16(Ctx& cx, const bf16* A, int lda, int K, int n_sl, Epi epi) {
    const int k_boxes = K >> 6;
    const uint32_t a_base = s_u32(A) + ((cx.lane & 15) * lda + (cx.lane >> 4) * 8) * 2;
    const bool active = cx.warp < n_sl;
    float acc[2][2][4];
    acc_zero(acc);
    for (int kb0 = 0; kb0 < k_boxes; kb0 += 2) mma_step(cx, a_base + kb0 * 128, min(2, k_boxes - kb0), active, acc);
    if (active) {
#pragma unroll
        for (int q = 0; q < 2; ++q) {
            const int j = q * 8 + 2 * cx.t;
            epi(cx.g, cx.warp, j, acc[q][0][0] + acc[q][1][0], acc[q][0][1] + acc[q][1][1]);
            epi(cx.g + 8, cx.warp, j, acc[q][0][2] + acc[q][1][2], acc[q][0][3] + acc[q][1][3]);
        }
    }
}

// GELU as the layer-by-layer GEMM epilogue computes it: x (1/2 + 1/2 tanh(x q(x^2))), q a quadratic fitted so that
// the result stays within 3e-5 of x Phi(x); one special-function instruction per element
__device__ __forceinline__ float gelu_fit(float v) {
    const float t = fminf(v * v, 50.f);                     // Phi has long saturated where the fitted q would turn over
    float q = fmaf(t, -3.5151945e-04f, 3.7005664e-02f);
    q = fmaf(q, t, 0.79750784f);
    float h;
    asm("tanh.approx.f32 %0, %1;" : "=f"(h) : "f"(v * q));
    return v * fmaf(h, 0.5f, 0.5f);
}

// abuf <- bf16(xres); stats[r] = (mean, rstd, 1/rstd) of the rounded row (what the tensor cores multiply).
// A warp takes two rows at once (two independent reduction chains); d is a multiple of 64, at most 384.
__device__ void round_rows_and_stats(Ctx& cx, int d, float eps) {
    const float* x = reinterpret_cast<const float*>(cx.sm + cx.L.xres);
    bf16* a = reinterpret_cast<bf16*>(cx.sm + cx.L.abuf);
    float4* st = reinterpret_cast<float4*>(cx.sm + cx.L.stats);
    const int n2 = d >> 6;                                  // float2 per lane and row
    for (int r = 2 * cx.warp; r < LT_ROWS; r += 2 * LT_CWARPS) {
        float2 v[2][6];
        float sum[2] = {0.f, 0.f};
#pragma unroll
        for (int q = 0; q < 2; ++q)
#pragma unroll
            for (int i = 0; i < 6; ++i) {
                v[q][i] = make_float2(0.f, 0.f);
                if (i < n2) {
                    const int c = 2 * cx.lane + 64 * i;
                    const float2 f = *reinterpret_cast<const float2*>(x + (r + q) * d + c);
                    const __nv_bfloat162 h = __floats2bfloat162_rn(f.x, f.y);
                    *reinterpret_cast<__nv_bfloat162*>(a + (r + q) * cx.L.lda + c) = h;
                    v[q][i] = __bfloat1622float2(h);
                    sum[q] += v[q][i].x + v[q][i].y;
                }
            }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            sum[0] += __shfl_xor_sync(0xFFFFFFFFu, sum[0], o);
            sum[1] += __shfl_xor_sync(0xFFFFFFFFu, sum[1], o);
        }
        const float inv_d = 1.f / (float)d;
        const float mean[2] = {sum[0] * inv_d, sum[1] * inv_d};
        float sq[2] = {0.f, 0.f};
#pragma unroll
        for (int q = 0; q < 2; ++q)
#pragma unroll
            for (int i = 0; i < 6; ++i)
                if (i < n2) { const float t0 = v[q][i].x - mean[q], t1 = v[q][i].y - mean[q]; sq[q] += t0 * t0 + t1 * t1; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            sq[0] += __shfl_xor_sync(0xFFFFFFFFu, sq[0], o);
            sq[1] += __shfl_xor_sync(0xFFFFFFFFu, sq[1], o);
        }
        if (cx.lane < 2) {
            const float rstd = rsqrtf((cx.lane ? sq[1] : sq[0]) * inv_d + eps);
            st[r + cx.lane] = make_float4(cx.lane ? mean[1] : mean[0], rstd, 1.f / rstd, 0.f);
        }
    }
}

__global__ void __launch_bounds__(LT_THREADS, 1) latency_forward_kernel(const __grid_constant__ LatArgs args) {
    extern __shared__ __align__(1024) uint8_t smem[];
    if (s_u32(smem) & 1023u) {                 // swizzled boxes need a 1024-byte aligned window
        if (threadIdx.x == 0) atomicCAS(args.status, 0, (int)PM_ERR_CUDA);
        return;
    }
    Ctx cx;
    cx.sm = smem;
    cx.L = lat_layout(args.d, args.mlp, args.patch_dim, args.tokens, args.layers, args.ring_slots);
    cx.ns = args.ring_slots;
    cx.warp = threadIdx.x >> 5; cx.lane = threadIdx.x & 31; cx.g = cx.lane >> 2; cx.t = cx.lane & 3;
    const int f = blockIdx.x / args.tiles_pf, rt = blockIdx.x % args.tiles_pf;     // slot, row tile
    const int frame = args.perm ? args.perm[f] : f;                                  // input / output row
    const int T = args.tokens, d = args.d, r0 = rt * LT_ROWS;
    const int tpad = (T + 15) / 16 * 16;
    const int rs = args.slabs_max * PM_SLAB;
    float* xres = reinterpret_cast<float*>(smem + cx.L.xres);
    bf16* abuf = reinterpret_cast<bf16*>(smem + cx.L.abuf);
    bf16* hbuf = reinterpret_cast<bf16*>(smem + cx.L.hbuf);
    bf16* qbuf = reinterpret_cast<bf16*>(smem + cx.L.qbuf);
    bf16* tbuf = reinterpret_cast<bf16*>(smem + cx.L.tbuf);
    const float4* stats = reinterpret_cast<const float4*>(smem + cx.L.stats);
    ActiveSet* as = reinterpret_cast<ActiveSet*>(smem + cx.L.misc);
    SlabTab* slabtab = reinterpret_cast<SlabTab*>(smem + cx.L.slabs);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + cx.L.misc + 192);
    cx.slot = 0; cx.phase = 0; cx.li = 0; cx.status = args.status; cx.abort_flag = abort_flag;
    if (threadIdx.x == 0) {
        for (int i = 0; i < LT_MAX_SLOTS; ++i) { bar_init(full_bar(cx, i), 1); bar_init(empty_bar(cx, i), LT_CWARPS); }
        bar_init(kfull_bar(cx), 1); bar_init(kempty_bar(cx), LT_CWARPS);
        bar_init(vfull_bar(cx), 1); bar_init(vempty_bar(cx), LT_CWARPS);
        for (int b = 0; b < 2; ++b) { bar_init(cfull_bar(cx, b), 1); bar_init(cempty_bar(cx, b), LT_CWARPS); }
        bar_init(kvdone_bar(cx, 0), LT_CWARPS); bar_init(kvdone_bar(cx, 1), LT_CWARPS);
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
    __syncthreads();
    // ---- per linear: the slabs of the set's adapters that touch it (adapters in ascending id; at most
    // LT_MAX_SLABS slabs, which the host checks against max_set * slabs_max)
    if ((int)threadIdx.x < args.layers * 4) {
        const LatLinear& lin = args.lin[threadIdx.x];
        SlabTab st;
        st.n = 0;
        if (lin.At) {
            for (int i = 0; i < as->n; ++i) {
                const int a = as->id[i];
                if (!((lin.adapted[a >> 5] >> (a & 31)) & 1u)) continue;
                for (int s = 0; s < as->slabs[i] && st.n < LT_MAX_SLABS; ++s) { st.who[st.n] = (uint8_t)i; st.sl[st.n] = (uint8_t)s; ++st.n; }
            }
        }
        slabtab[threadIdx.x] = st;
    }
    __syncthreads();
    // ---- the weight producer: one thread, the whole network's static operands in consumption order
    if (cx.warp == LT_CWARPS) {
        if (cx.lane != 0) return;
        SlabTab none;
        none.n = 0;
        produce_linear(cx, args.lin + (size_t)args.layers * 4, none, *as, rs, args.slabs_max, d, false);
        for (int l = 0; l < args.layers && !*abort_flag; ++l)
            for (int j = 0; j < 4; ++j)
                produce_linear(cx, args.lin + (size_t)l * 4 + j, slabtab[l * 4 + j], *as, rs, args.slabs_max, d, j == 0);
        return;
    }
    // ---- the key/value producer: per block, wait for the frame's CTAs, then one head after the other
    if (cx.warp == LT_CWARPS + 1) {
        if (cx.lane != 0) return;
        uint32_t idx = 0;
        for (int l = 0; l < args.layers && !*abort_flag; ++l) {
            // Twice per block -- for the first head, then for the others -- : the consumer warps have stored this
            // CTA's keys and values (ordinary stores, fetched by TMA on the other side: order the two proxies as
            // well as the scopes), so the CTA counts itself in: everything its threads stored up to there is
            // visible to whoever sees the count.  Then the heads' keys and values, one after the other.
            const int kv_row0 = ((l & 1) * args.n_frames + f) * T;
            const bool two = chunk_order(3 * d, d, true).reorder;   // else: one count-in per block
            for (int part = 0; part < (two ? 2 : 1) && !*abort_flag; ++part) {
                bar_wait(cx, kvdone_bar(cx, two ? part : 1), (uint32_t)l & 1u);
                if (*abort_flag) break;
                asm volatile("fence.proxy.async.global;" ::: "memory");
                __threadfence();
                atomicAdd(args.bar + f, 1u);
                const unsigned int per = two ? 2u : 1u;
                const unsigned int want = (unsigned int)args.tiles_pf * (per * (unsigned int)l + (unsigned int)part + 1u);
                const long long t0 = clock64();
                unsigned int seen;
                do {
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(args.bar + f) : "memory");
                    if (seen < want && (*abort_flag || clock64() - t0 > LT_WAIT_CYCLES)) {
                        if (!*abort_flag) { *abort_flag = 1; atomicCAS(args.status, 0, (int)PM_ERR_TIMEOUT); }
                        break;
                    }
                } while (seen < want);
                if (*abort_flag) break;
                asm volatile("fence.proxy.async.global;" ::: "memory");
                const int h0 = !two ? 0 : part == 0 ? 0 : 1, h1 = !two ? args.heads : part == 0 ? 1 : args.heads;
                for (int h = h0; h < h1; ++h, ++idx) {
                    bar_wait(cx, kempty_bar(cx), (idx & 1u) ^ 1u);
                    bar_expect(kfull_bar(cx), (uint32_t)tpad * 128u);
                    tma_box(s_u32(smem + cx.L.kbuf), &args.tm_kv, h * LT_HD, kv_row0, kfull_bar(cx));
                    bar_wait(cx, vempty_bar(cx), (idx & 1u) ^ 1u);
                    bar_expect(vfull_bar(cx), (uint32_t)tpad * 128u);
                    tma_box(s_u32(smem + cx.L.vbuf), &args.tm_kv, d + h * LT_HD, kv_row0, vfull_bar(cx));
                }
            }
        }
        return;
    }

    // ================================ consumers (256 threads) ================================
    // ---- patch gather: hbuf[r][c*P*P + py*P + px] = frame[c][gy*P + py][gx*P + px] of token r0 + r (token 0 = CLS)
    {
        const int P = 16, per_row = args.patch_dim / 8;
        const bf16* fr = args.frames + (size_t)frame * 3 * args.img * args.img;
        for (int i = threadIdx.x; i < LT_ROWS * per_row; i += LT_CTHREADS) {
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
    // the kilobyte behind the values is read as keys whose probabilities are zero: it has to hold finite numbers
    for (int i = threadIdx.x; i < 256; i += LT_CTHREADS)
        reinterpret_cast<uint32_t*>(smem + cx.L.vbuf + cx.L.kv_bytes - 1024)[i] = 0u;
    consumer_sync();

    // the vector pack of the linear the consumers are at: wait for it / hand its buffer back
    auto pack_acquire = [&]() -> const float* {
        bar_wait(cx, cfull_bar(cx, cx.li & 1u), (cx.li >> 1) & 1u);
        return reinterpret_cast<const float*>(smem + cx.L.colv) + (cx.li & 1u) * cx.L.cv_floats;
    };
    auto pack_release = [&]() {
        __syncwarp();
        if (cx.lane == 0) bar_arrive(cempty_bar(cx, cx.li & 1u));
        ++cx.li;
    };
    // ---- patch projection + positions; the CLS row
    {
        const float* cv = pack_acquire();
        linear16(cx, hbuf, cx.L.ldh, args.patch_dim, d, 0, d, false, [&](int n0, float (&y)[2][4]) {
#pragma unroll
            for (int hi = 0; hi < 2; ++hi) {
                const int r = cx.g + 8 * hi, tok = r0 + r;
                float2 p[2] = {make_float2(0.f, 0.f), make_float2(0.f, 0.f)};
                if (tok < T) {
#pragma unroll
                    for (int q = 0; q < 2; ++q) p[q] = *reinterpret_cast<const float2*>(args.pos + (size_t)tok * d + n0 + 8 * q);
                }
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int n = n0 + 8 * q;
                    float2 out = make_float2(0.f, 0.f);             // rows past the frame stay zero
                    if (tok == 0) out = make_float2(args.cls[n] + p[q].x, args.cls[n + 1] + p[q].y);
                    else if (tok < T) out = make_float2(y[q][2 * hi] + cv[n] + p[q].x, y[q][2 * hi + 1] + cv[n + 1] + p[q].y);
                    *reinterpret_cast<float2*>(xres + r * d + n) = out;
                }
            }
        });
        pack_release();
    }
    consumer_sync();

    // LoRA shrink of a linear with slab table `st` on the rows A: t[r][16 i + j] (bf16) = s_a (x A_a)
    // (folded linears: s_a ((x A' - mean c1) + c2 / rstd), the fused accumulator being scaled by rstd afterwards)
    auto shrink = [&](const SlabTab& st, const bf16* A, int lda, int K, int N, bool folded, const float* cv) {
        if (!st.n) return;
        shrink16(cx, A, lda, K, st.n, [&](int r, int i, int j, float v0, float v1) {
            if (folded) {
                const float* c1 = cv + 2 * N + i * PM_SLAB + j;
                const float* c2 = c1 + LT_MAX_SLABS * PM_SLAB;
                v0 = (v0 - stats[r].x * c1[0]) + c2[0] * stats[r].z;
                v1 = (v1 - stats[r].x * c1[1]) + c2[1] * stats[r].z;
            }
            const float sc = as->scale[st.who[i]];
            *reinterpret_cast<uint32_t*>(tbuf + r * cx.L.ldt + i * PM_SLAB + j) = pk_bf16(v0 * sc, v1 * sc);
        });
        consumer_sync();
    };
    auto residual = [&](const float* cv) {
        return [=](int n0, float (&y)[2][4]) {
            float2 x[2][2], b[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                b[q] = *reinterpret_cast<const float2*>(cv + n0 + 8 * q);
                x[q][0] = *reinterpret_cast<const float2*>(xres + cx.g * d + n0 + 8 * q);
                x[q][1] = *reinterpret_cast<const float2*>(xres + (cx.g + 8) * d + n0 + 8 * q);
            }
#pragma unroll
            for (int q = 0; q < 2; ++q)
#pragma unroll
                for (int hi = 0; hi < 2; ++hi)
                    if (r0 + cx.g + 8 * hi < T)
                        *reinterpret_cast<float2*>(xres + (cx.g + 8 * hi) * d + n0 + 8 * q) =
                            make_float2(x[q][hi].x + y[q][2 * hi] + b[q].x, x[q][hi].y + y[q][2 * hi + 1] + b[q].y);
        };
    };

    const float att_scale = 0.125f * 1.4426950408889634f;  // 1/sqrt(64) * log2(e)
    uint32_t head_no = 0;                                    // heads attended so far (all blocks)
    for (int l = 0; l < args.layers; ++l) {
        const SlabTab* st = slabtab + l * 4;
        bf16* kvb = args.kv + (size_t)(l & 1) * args.n_frames * T * 2 * d + (size_t)f * T * 2 * d;
        // ---- qkv (LayerNorm 1 folded): q stays here, k and v go to the frame's exchange buffer
        round_rows_and_stats(cx, d, args.eps);
        consumer_sync();
        {
            const float* cv = pack_acquire();
            shrink(st[0], abuf, cx.L.lda, d, 3 * d, true, cv);
            const float4 s_lo = stats[cx.g], s_hi = stats[cx.g + 8];
            linear16(cx, abuf, cx.L.lda, d, 3 * d, st[0].n, d, true, [&](int n0, float (&y)[2][4]) {
                float2 b[2], gs[2];
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    b[q] = *reinterpret_cast<const float2*>(cv + n0 + 8 * q);
                    gs[q] = *reinterpret_cast<const float2*>(cv + 3 * d + n0 + 8 * q);
                }
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int n = n0 + 8 * q;
                    const uint32_t lo = pk_bf16(s_lo.y * (y[q][0] - s_lo.x * gs[q].x) + b[q].x, s_lo.y * (y[q][1] - s_lo.x * gs[q].y) + b[q].y);
                    const uint32_t hi = pk_bf16(s_hi.y * (y[q][2] - s_hi.x * gs[q].x) + b[q].x, s_hi.y * (y[q][3] - s_hi.x * gs[q].y) + b[q].y);
                    if (n < d) {
                        *reinterpret_cast<uint32_t*>(qbuf + cx.g * cx.L.ldq + n) = lo;
                        *reinterpret_cast<uint32_t*>(qbuf + (cx.g + 8) * cx.L.ldq + n) = hi;
                    } else {
                        if (r0 + cx.g < T) *reinterpret_cast<uint32_t*>(kvb + (size_t)(r0 + cx.g) * 2 * d + (n - d)) = lo;
                        if (r0 + cx.g + 8 < T) *reinterpret_cast<uint32_t*>(kvb + (size_t)(r0 + cx.g + 8) * 2 * d + (n - d)) = hi;
                    }
                }
            });
            pack_release();
        }
        consumer_sync();                                     // all of q is in place
        // ---- attention, head by head.  Warp w: key range w / 2 of four, dims 32 (w % 2) .. + 31 of the head.
        // Keys and values of a head are one TMA box each ([tpad rows][64 dims], 128B swizzle; rows past the
        // frame hold a neighbour's rows or zeros and are masked below).
        {
            const int kr = cx.warp >> 1, dh = cx.warp & 1;
            const int n_t8 = tpad / 8;
            const int t8_lo = (n_t8 * kr) / LT_KSPLIT, t8_hi = (n_t8 * (kr + 1)) / LT_KSPLIT, n_t = t8_hi - t8_lo;   // <= LT_ST tiles
            // a key tile is 8 rows of 128 bytes, so a lane's row keeps its swizzle phase (lane & 7) from tile
            // to tile: one address per k16 step (keys) or pair of dim tiles (values), plus a multiple of 1 KB
            const int l7 = cx.lane & 7, mi = cx.lane >> 3;
            uint32_t k_addr[2], v_addr[2];
#pragma unroll
            for (int kp = 0; kp < 2; ++kp)                   // one fetch brings a tile's keys for two k16 steps (32 dims)
                k_addr[kp] = s_u32(smem + cx.L.kbuf) + (t8_lo * 8 + l7) * 128 + (((kp * 4 + mi) ^ l7) << 4);
#pragma unroll
            for (int n = 0; n < 2; ++n)
                v_addr[n] = s_u32(smem + cx.L.vbuf) + (t8_lo * 8 + (mi & 1) * 8 + l7) * 128 + (((dh * 4 + n * 2 + (mi >> 1)) ^ l7) << 4);
            float* part = reinterpret_cast<float*>(smem + cx.L.hbuf);
            for (int h = 0; h < args.heads; ++h, ++head_no) {
                uint32_t qa[4][4];
#pragma unroll
                for (int ks = 0; ks < 4; ++ks)
                    ldsm4(s_u32(qbuf) + ((cx.lane & 15) * cx.L.ldq + h * LT_HD + ks * 16 + (cx.lane >> 4) * 8) * 2,
                          qa[ks][0], qa[ks][1], qa[ks][2], qa[ks][3]);
                bar_wait(cx, kfull_bar(cx), head_no & 1u);
                float s[LT_ST][4];
#pragma unroll
                for (int j = 0; j < LT_ST; ++j) s[j][0] = s[j][1] = s[j][2] = s[j][3] = 0.f;
                // tile by tile inside each k16 step: consecutive multiplications go to different accumulators
#pragma unroll
                for (int kp = 0; kp < 2; ++kp) {
                    uint32_t kf[LT_ST][4];
#pragma unroll
                    for (int j = 0; j < LT_ST; ++j)
                        if (j < n_t) ldsm4(k_addr[kp] + j * 1024, kf[j][0], kf[j][1], kf[j][2], kf[j][3]);
#pragma unroll
                    for (int j = 0; j < LT_ST; ++j)
                        if (j < n_t) mma16816(s[j], qa[2 * kp], kf[j][0], kf[j][1]);
#pragma unroll
                    for (int j = 0; j < LT_ST; ++j)
                        if (j < n_t) mma16816(s[j], qa[2 * kp + 1], kf[j][2], kf[j][3]);
                }
                __syncwarp();
                if (cx.lane == 0) bar_arrive(kempty_bar(cx));        // the next head's keys may land
                float m_lo = -INFINITY, m_hi = -INFINITY;
#pragma unroll
                for (int j = 0; j < LT_ST; ++j) {
                    const int key = (t8_lo + j) * 8 + 2 * cx.t;
                    if (j >= n_t || (t8_lo + j) * 8 + 8 > T) {       // only the frame's last tile has keys to mask
#pragma unroll
                        for (int e = 0; e < 4; ++e)
                            if (!(j < n_t && key + (e & 1) < T)) s[j][e] = -INFINITY;
                    }
                    m_lo = fmaxf(m_lo, fmaxf(s[j][0], s[j][1]));
                    m_hi = fmaxf(m_hi, fmaxf(s[j][2], s[j][3]));
                }
                m_lo = fmaxf(m_lo, __shfl_xor_sync(0xFFFFFFFFu, m_lo, 1));
                m_lo = fmaxf(m_lo, __shfl_xor_sync(0xFFFFFFFFu, m_lo, 2));
                m_hi = fmaxf(m_hi, __shfl_xor_sync(0xFFFFFFFFu, m_hi, 1));
                m_hi = fmaxf(m_hi, __shfl_xor_sync(0xFFFFFFFFu, m_hi, 2));
                // the maxima in the exponent's units (1/sqrt(64) log2 e); a warp whose keys are all beyond the
                // frame contributes nothing (its maximum stays -inf)
                m_lo *= att_scale; m_hi *= att_scale;
                const float ms_lo = m_lo == -INFINITY ? 0.f : m_lo, ms_hi = m_hi == -INFINITY ? 0.f : m_hi;
                float l_lo = 0.f, l_hi = 0.f;
                uint32_t pa[LT_ST / 2][4];
#pragma unroll
                for (int j = 0; j < LT_ST; ++j) {
                    const float p0 = ex2(fmaf(s[j][0], att_scale, -ms_lo)), p1 = ex2(fmaf(s[j][1], att_scale, -ms_lo));
                    const float p2 = ex2(fmaf(s[j][2], att_scale, -ms_hi)), p3 = ex2(fmaf(s[j][3], att_scale, -ms_hi));
                    l_lo += p0 + p1;
                    l_hi += p2 + p3;
                    pa[j >> 1][(j & 1) * 2 + 0] = pk_bf16(p0, p1);
                    pa[j >> 1][(j & 1) * 2 + 1] = pk_bf16(p2, p3);
                }
                l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 1);
                l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 2);
                l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 1);
                l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 2);
                float o[4][4];
#pragma unroll
                for (int i = 0; i < 4; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
                bar_wait(cx, vfull_bar(cx), head_no & 1u);
                // 16-key steps of this warp's keys.  The second tile of the last step may belong to the next
                // range (its probabilities are 0 here) or lie behind the last key (the kilobyte of zeros)
#pragma unroll
                for (int kk = 0; kk < LT_ST / 2; ++kk) {
                    if (2 * kk < n_t) {
#pragma unroll
                        for (int n = 0; n < 2; ++n) {            // pairs of 8-dim tiles
                            uint32_t b0, b1, b2, b3;
                            ldsm4t(v_addr[n] + kk * 2048, b0, b1, b2, b3);
                            mma16816(o[2 * n], pa[kk], b0, b1);
                            mma16816(o[2 * n + 1], pa[kk], b2, b3);
                        }
                    }
                }
                __syncwarp();
                if (cx.lane == 0) bar_arrive(vempty_bar(cx));
                // partial results: part[range][row][0..63] = o, [64] = max, [65] = sum
                float* pw = part + (size_t)kr * LT_ROWS * (LT_HD + 2);
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int c = dh * 32 + i * 8 + 2 * cx.t;
                    *reinterpret_cast<float2*>(pw + cx.g * (LT_HD + 2) + c) = make_float2(o[i][0], o[i][1]);
                    *reinterpret_cast<float2*>(pw + (cx.g + 8) * (LT_HD + 2) + c) = make_float2(o[i][2], o[i][3]);
                }
                if (dh == 0 && cx.t == 0) {
                    pw[cx.g * (LT_HD + 2) + 64] = m_lo; pw[cx.g * (LT_HD + 2) + 65] = l_lo;
                    pw[(cx.g + 8) * (LT_HD + 2) + 64] = m_hi; pw[(cx.g + 8) * (LT_HD + 2) + 65] = l_hi;
                }
                consumer_sync();
                {   // merge: thread -> (row, four dims)
                    const int r = threadIdx.x >> 4, c4 = (threadIdx.x & 15) * 4;
                    float m = -INFINITY;
#pragma unroll
                    for (int w = 0; w < LT_KSPLIT; ++w) m = fmaxf(m, part[(w * LT_ROWS + r) * (LT_HD + 2) + 64]);
                    float den = 0.f, num[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int w = 0; w < LT_KSPLIT; ++w) {
                        const float* pr = part + (w * LT_ROWS + r) * (LT_HD + 2);
                        const float e = pr[64] == -INFINITY ? 0.f : ex2(pr[64] - m);
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
                consumer_sync();
            }
        }
        // ---- proj (+ residual)
        {
            const float* cv = pack_acquire();
            shrink(st[1], abuf, cx.L.lda, d, d, false, cv);
            linear16(cx, abuf, cx.L.lda, d, d, st[1].n, d, false, residual(cv));
            pack_release();
        }
        consumer_sync();
        // ---- fc1 (LayerNorm 2 folded, GELU) and fc2 (+ residual)
        round_rows_and_stats(cx, d, args.eps);
        consumer_sync();
        {
            const float* cv = pack_acquire();
            const int N = args.mlp;
            shrink(st[2], abuf, cx.L.lda, d, N, true, cv);
            const float4 s_lo = stats[cx.g], s_hi = stats[cx.g + 8];
            linear16(cx, abuf, cx.L.lda, d, N, st[2].n, d, false, [&](int n0, float (&y)[2][4]) {
                float2 b[2], gs[2];
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    b[q] = *reinterpret_cast<const float2*>(cv + n0 + 8 * q);
                    gs[q] = *reinterpret_cast<const float2*>(cv + N + n0 + 8 * q);
                }
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const int n = n0 + 8 * q;
                    *reinterpret_cast<uint32_t*>(hbuf + cx.g * cx.L.ldh + n) =
                        pk_bf16(gelu_fit(s_lo.y * (y[q][0] - s_lo.x * gs[q].x) + b[q].x), gelu_fit(s_lo.y * (y[q][1] - s_lo.x * gs[q].y) + b[q].y));
                    *reinterpret_cast<uint32_t*>(hbuf + (cx.g + 8) * cx.L.ldh + n) =
                        pk_bf16(gelu_fit(s_hi.y * (y[q][2] - s_hi.x * gs[q].x) + b[q].x), gelu_fit(s_hi.y * (y[q][3] - s_hi.x * gs[q].y) + b[q].y));
                }
            });
            pack_release();
        }
        consumer_sync();
        {
            const float* cv = pack_acquire();
            shrink(st[3], hbuf, cx.L.ldh, args.mlp, d, false, cv);
            linear16(cx, hbuf, cx.L.ldh, args.mlp, d, st[3].n, d, false, residual(cv));
            pack_release();
        }
        consumer_sync();
    }

    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);     // copies still in flight land before shared memory goes away
        return;
    }
    if (rt != 0) return;

    // ---- heads on the CLS row (row 0 of the frame's first CTA): final LayerNorm, base head, adapter heads
    float* z = reinterpret_cast<float*>(smem + cx.L.hbuf);
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
    for (int k = threadIdx.x; k < args.n_classes; k += LT_CTHREADS) srow[k] = 0.f;
    consumer_sync();
    // one thread per head row: its d weights are independent 16-byte loads, all in flight at once
    auto dot = [&](const bf16* w) {
        float acc0 = 0.f, acc1 = 0.f;
        for (int c = 0; c < d; c += 8) {
            const uint4 u = __ldg(reinterpret_cast<const uint4*>(w + c));
            const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                acc0 = fmaf(z[c + 2 * q], __bfloat162float(h2[q].x), acc0);
                acc1 = fmaf(z[c + 2 * q + 1], __bfloat162float(h2[q].y), acc1);
            }
        }
        return acc0 + acc1;
    };
    if (args.base_out) {
        for (int k = threadIdx.x; k < args.n_classes; k += LT_CTHREADS) {
            const float v = dot(args.head_wt + (size_t)k * d) + args.head_b[k];
            args.base_out[(size_t)frame * args.n_classes + k] = 1.f / (1.f + expf(-v));
        }
    }
    for (int i = 0; i < as->n; ++i) {
        const int a = as->id[i];
        for (int r = args.hoff[a] + threadIdx.x; r < args.hoff[a + 1]; r += LT_CTHREADS) {
            const float v = dot(args.hcat + (size_t)r * d) + args.hbias[r];
            // scores are positive: the maximum over adapters is an integer maximum of the bit patterns
            atomicMax(reinterpret_cast<int*>(srow + args.hcls[r]), __float_as_int(1.f / (1.f + expf(-v))));
        }
    }
}

// the most ring slots that fit beside everything else (0: the geometry does not fit at all)
int lat_ring_slots(int d, int mlp, int patch_dim, int tokens, int layers) {
    const int fixed = lat_layout(d, mlp, patch_dim, tokens, layers, 0).total;
    const int room = 227 * 1024 - fixed;
    if (room < 2 * LT_SLOT_BYTES) return 0;
    return room / LT_SLOT_BYTES < LT_MAX_SLOTS ? room / LT_SLOT_BYTES : LT_MAX_SLOTS;
}

}  // namespace

size_t latency_smem_bytes(int d, int mlp, int patch_dim, int tokens, int layers) {
    const int slots = lat_ring_slots(d, mlp, patch_dim, tokens, layers);
    if (!slots) return (size_t)1 << 30;
    return (size_t)lat_layout(d, mlp, patch_dim, tokens, layers, slots).total;
}

cudaError_t launch_latency_forward(const Launch& L, const LatArgs& a) {
    const int slots = lat_ring_slots(a.d, a.mlp, a.patch_dim, a.tokens, a.layers);
    if (!slots || a.layers * 4 > LT_THREADS) return cudaErrorInvalidValue;
    const size_t smem = (size_t)lat_layout(a.d, a.mlp, a.patch_dim, a.tokens, a.layers, slots).total;
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
    copy.ring_slots = slots;
    // the frames' arrival counters start at zero (an aborted launch may have left them anywhere)
    cudaError_t e = cudaMemsetAsync(a.bar, 0, sizeof(unsigned int) * a.n_frames, L.st);
    if (e != cudaSuccess) return e;
    e = cudaLaunchKernelEx(&cfg, latency_forward_kernel, copy);
    BUMP(L);
    return e != cudaSuccess ? e : cudaGetLastError();
}
