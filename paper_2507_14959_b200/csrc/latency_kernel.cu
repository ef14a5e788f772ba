// Whole-network kernel for a handful of frames (the single-stream operating point of Sec. 4): patch
// embedding, all encoder blocks with their unmerged LoRA terms (Sec. 3.1), final LayerNorm, base and
// adapter heads with sigmoid and merge (Fig. 5b) in ONE launch.
//
// Everything in a ViT block except attention is local to a token row, so a CTA owns 16 token rows of one
// frame from the first layer to the last and keeps their residual stream (fp32) and every intermediate in
// shared memory; the weights stream through shared memory (cp.async, two stages) and are the only thing
// read from L2 -- every CTA reads all of them, which is what bounds a frame's latency.  The one exchange
// per block is attention: each CTA publishes the keys and values of its rows (two global buffers used in
// turn), the CTAs of a frame meet at a counter (bounded wait), then each CTA attends from its 16 query rows
// to all keys of its frame, head by head (the eight warps split the keys and merge their partial softmax
// results).  Contractions run on mma.sync m16n8k16 (bf16 in, fp32 accumulate): with 16 rows per CTA there is
// no 128-row tile to give to tcgen05, and the tensor work is a small part of the time anyway.
// LayerNorm uses the folded form the other kernels use: y = rstd (x W' - mean g) + b'.
#include "common.cuh"

#define BUMP(L) do { if ((L).launches) ++*(L).launches; } while (0)

namespace {

constexpr int LT_ROWS = 16;
constexpr int LT_THREADS = 256;
constexpr int LT_WARPS = 8;
constexpr int LT_KB = 192;                 // K columns of a weight stage
constexpr int LT_WSTRIDE = LT_KB + 8;      // bf16 per staged weight row (16-byte skew: conflict-free ldmatrix)
constexpr int LT_NCHUNK = 64;              // output columns per stage: one n8 tile per warp
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

}  // namespace

namespace {

struct LatSmem {               // offsets (bytes) into dynamic shared memory
    int xres, abuf, hbuf, qbuf, tbuf, stats, region, part, misc, total;
    int lda, ldh, ldq, ldt;    // row strides in bf16 elements
};

__host__ __device__ inline LatSmem lat_layout(int d, int mlp, int patch_dim, int rs_total, int tokens) {
    LatSmem s;
    auto up = [](int v) { return (v + 127) & ~127; };
    s.lda = d + 8; s.ldh = (mlp > patch_dim ? mlp : patch_dim) + 8; s.ldq = d + 8; s.ldt = rs_total + 8;
    int o = 0;
    s.xres = o; o = up(o + LT_ROWS * d * 4);
    s.abuf = o; o = up(o + LT_ROWS * s.lda * 2);
    s.hbuf = o; o = up(o + LT_ROWS * s.ldh * 2);
    s.qbuf = o; o = up(o + LT_ROWS * s.ldq * 2);
    s.tbuf = o; o = up(o + LT_ROWS * s.ldt * 2);
    s.stats = o; o = up(o + LT_ROWS * 16);
    // weight stages (2 x 64 rows) or one head's keys and values (2 x tpad rows of 128 bytes)
    const int tpad = (tokens + 15) / 16 * 16;
    const int wbytes = 2 * LT_NCHUNK * LT_WSTRIDE * 2, kvbytes = 2 * tpad * 128;
    s.region = o; o = up(o + (wbytes > kvbytes ? wbytes : kvbytes));
    s.part = o; o = up(o + LT_WARPS * LT_ROWS * (LT_HD + 2) * 4);      // partial attention results of the warps
    s.misc = o; o = up(o + 256);
    s.total = o;
    return s;
}

struct Ctx {
    uint8_t* sm;
    LatSmem L;
    int warp, lane, g, t;
};

// Streams W^T rows [n0, n0 + 64) x columns [k0, k0 + len) into stage `buf` (rows past n_out are skipped:
// their products are never used).
__device__ __forceinline__ void stage_weights(const Ctx& cx, int buf, const bf16* Wt, int N, int K, int n0, int k0, int len) {
    const int chunks = len >> 3;                     // 16-byte pieces per row
    const uint32_t dst0 = s_u32(cx.sm + cx.L.region) + buf * (LT_NCHUNK * LT_WSTRIDE * 2);
    for (int i = threadIdx.x; i < LT_NCHUNK * chunks; i += LT_THREADS) {
        const int r = i / chunks, c = i % chunks;
        if (n0 + r < N) cp16(dst0 + (r * LT_WSTRIDE + c * 8) * 2, Wt + (size_t)(n0 + r) * K + k0 + c * 8);
    }
}

struct LoraExp {               // LoRA expand of the current linear: t (shared memory) times B slabs (global)
    int n_act;
    int adapter[LT_MAX_SET], slabs[LT_MAX_SET];
    const bf16* Bt;
    int slabs_max, rs;         // rs: columns of t per adapter
};

// y[16, N] = A[16, K] W + LoRA expand, handed element-wise to epi(row, n, value).  A: bf16 in shared memory
// with row stride lda.  All threads of the CTA call it.
template <typename Epi>
__device__ void linear16(const Ctx& cx, const bf16* A, int lda, const bf16* Wt, int N, int K, const LoraExp* lx, Epi epi) {
    const int n_chunks = (N + LT_NCHUNK - 1) / LT_NCHUNK, k_blocks = (K + LT_KB - 1) / LT_KB;
    const int total = n_chunks * k_blocks;
    const uint32_t a_base = s_u32(A), w_base = s_u32(cx.sm + cx.L.region), t_base = s_u32(cx.sm + cx.L.tbuf);
    const int lane = cx.lane, warp = cx.warp;
    stage_weights(cx, 0, Wt, N, K, 0, 0, min(LT_KB, K));
    cp_commit();
    float acc[4] = {0.f, 0.f, 0.f, 0.f};
    for (int it = 0; it < total; ++it) {
        const int nc = it / k_blocks, kb = it % k_blocks;
        if (it + 1 < total) {
            const int nc1 = (it + 1) / k_blocks, kb1 = (it + 1) % k_blocks;
            stage_weights(cx, (it + 1) & 1, Wt, N, K, nc1 * LT_NCHUNK, kb1 * LT_KB, min(LT_KB, K - kb1 * LT_KB));
            cp_commit();
            cp_wait<1>();
        } else {
            cp_wait<0>();
        }
        __syncthreads();
        const int n8 = nc * LT_NCHUNK + warp * 8;
        const bool active = n8 < N;
        if (kb == 0) { acc[0] = acc[1] = acc[2] = acc[3] = 0.f; }
        if (active) {
            const int k0 = kb * LT_KB, len = min(LT_KB, K - k0);
            const uint32_t a_row = a_base + ((lane & 15) * lda + k0 + (lane >> 4) * 8) * 2;
            const uint32_t w_row = w_base + (it & 1) * (LT_NCHUNK * LT_WSTRIDE * 2) +
                                   ((warp * 8 + (lane & 7)) * LT_WSTRIDE + ((lane >> 3) & 1) * 8) * 2;
            for (int kk = 0; kk < len; kk += 16) {
                uint32_t a[4], b0, b1;
                ldsm4(a_row + kk * 2, a[0], a[1], a[2], a[3]);
                ldsm2(w_row + kk * 2, b0, b1);
                mma16816(acc, a, b0, b1);
            }
            if (kb == k_blocks - 1) {
                if (lx) {
                    for (int p = 0; p < lx->n_act; ++p)
                        for (int s = 0; s < lx->slabs[p]; ++s) {
                            uint32_t a[4];
                            ldsm4(t_base + ((lane & 15) * cx.L.ldt + p * lx->rs + s * 16 + (lane >> 4) * 8) * 2, a[0], a[1], a[2], a[3]);
                            const bf16* bp = lx->Bt + (((size_t)(lx->adapter[p] * lx->slabs_max + s) * N) + n8 + cx.g) * PM_SLAB;
                            const uint32_t b0 = __ldg(reinterpret_cast<const unsigned int*>(bp + 2 * cx.t));
                            const uint32_t b1 = __ldg(reinterpret_cast<const unsigned int*>(bp + 2 * cx.t + 8));
                            mma16816(acc, a, b0, b1);
                        }
                }
                const int n = n8 + 2 * cx.t;
                epi(cx.g, n, acc[0]); epi(cx.g, n + 1, acc[1]);
                epi(cx.g + 8, n, acc[2]); epi(cx.g + 8, n + 1, acc[3]);
            }
        }
        __syncthreads();          // the stage may be overwritten two iterations from now
    }
}

__device__ __forceinline__ float gelu_exact(float v) { return 0.5f * v * (1.f + erff(v * 0.70710678118654752440f)); }

// abuf <- bf16(xres); stats[r] = (mean, rstd, 1/rstd) of the rounded row (what the tensor cores multiply)
__device__ void round_rows_and_stats(const Ctx& cx, int d, float eps) {
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
__device__ void lora_shrink(const Ctx& cx, const LatLinear& lin, const ActiveSet& as, int slabs_max, const bf16* A, int lda,
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
        linear16(cx, A, lda, lin.At + (size_t)a * lx->rs * lin.k_in, rs_a, lin.k_in, nullptr,
                 [&](int r, int j, float v) {
                     if (folded) v = (v - st[r].x * c1[j]) + c2[j] * st[r].z;
                     tb[r * ldt + col0 + j] = __float2bfloat16_rn(v * sc);
                 });
    }
    __syncthreads();
}

__global__ void __launch_bounds__(LT_THREADS, 1) latency_forward_kernel(const LatArgs args) {
    extern __shared__ __align__(128) uint8_t smem[];
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
    linear16(cx, hbuf, cx.L.ldh, args.patch.Wt, d, args.patch_dim, nullptr, [&](int r, int n, float v) {
        const int tok = r0 + r;
        float out = 0.f;
        if (tok == 0) out = args.cls[n] + args.pos[n];
        else if (tok < T) out = v + args.patch.bias[n] + args.pos[(size_t)tok * d + n];
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
            linear16(cx, abuf, cx.L.lda, lin[0].Wt, 3 * d, d, lx.n_act ? &lx : nullptr, [&](int r, int n, float v) {
                const float y = stats[r].y * (v - stats[r].x * lg[n]) + bb[n];
                if (n < d) qbuf[r * cx.L.ldq + n] = __float2bfloat16_rn(y);
                else if (r0 + r < T) kvb[(size_t)(r0 + r) * 2 * d + (n - d)] = __float2bfloat16_rn(y);
            });
        }
        // ---- the CTAs of the frame meet: all keys and values of this block are in place
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
        for (int h = 0; h < args.heads; ++h) {
            uint8_t* Ks = smem + cx.L.region;
            uint8_t* Vs = Ks + tpad * 128;
            for (int i = threadIdx.x; i < tpad * 16; i += LT_THREADS) {
                const int r = i >> 4, c = i & 7, isv = (i >> 3) & 1;
                uint8_t* dst = (isv ? Vs : Ks) + r * 128 + ((c ^ (r & 7)) << 4);
                if (r < T) cp16(s_u32(dst), kvb + (size_t)r * 2 * d + isv * d + h * LT_HD + c * 8);
                else *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
            }
            cp_commit();
            cp_wait<0>();
            __syncthreads();
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
            linear16(cx, abuf, cx.L.lda, lin[1].Wt, d, d, lx.n_act ? &lx : nullptr,
                     [&](int r, int n, float v) { if (r0 + r < T) xres[r * d + n] += v + bb[n]; });
        }
        __syncthreads();
        // ---- fc1 (LayerNorm 2 folded, GELU) and fc2 (+ residual)
        round_rows_and_stats(cx, d, args.eps);
        __syncthreads();
        lora_shrink(cx, lin[2], aset, args.slabs_max, abuf, cx.L.lda, &lx);
        {
            const float* lg = lin[2].ln_g; const float* bb = lin[2].bias;
            linear16(cx, abuf, cx.L.lda, lin[2].Wt, args.mlp, d, lx.n_act ? &lx : nullptr, [&](int r, int n, float v) {
                hbuf[r * cx.L.ldh + n] = __float2bfloat16_rn(gelu_exact(stats[r].y * (v - stats[r].x * lg[n]) + bb[n]));
            });
        }
        __syncthreads();
        lora_shrink(cx, lin[3], aset, args.slabs_max, hbuf, cx.L.ldh, &lx);
        {
            const float* bb = lin[3].bias;
            linear16(cx, hbuf, cx.L.ldh, lin[3].Wt, d, args.mlp, lx.n_act ? &lx : nullptr,
                     [&](int r, int n, float v) { if (r0 + r < T) xres[r * d + n] += v + bb[n]; });
        }
        __syncthreads();
    }

    if (rt != 0 || *abort_flag) return;

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
