// Attention of the bf16 build: softmax(q k^T / 8) v per (frame, head), head dim 64.
//
// Three kernels.  The two that serve the model shapes, attention_pipe_kernel (one key block, up to
// 208 tokens: persistent, two query tiles in flight) and attention_tc_kernel (up to 624 tokens, several
// key blocks), run both contractions on the tcgen05 tensor cores with scores and probabilities in
// tensor memory; they are described where they are defined.  attention_mma_kernel is the
// register-level kernel for sequences beyond 624 tokens:
//
// One CTA owns one (frame, head) (or a slice of its query rows when there are more than 256):
// K and V of the head are staged once in shared memory (16-byte chunks XOR-swizzled by row so
// that ldmatrix is conflict-free), each warp owns 16 query rows and walks the keys in blocks of
// 64 with an online softmax in fp32; both contractions run on the tensor cores
// (mma.sync m16n8k16, bf16 in, fp32 accumulate).  Key blocks are trimmed to the 8-key tile, so
// 197 tokens cost 200 key columns, not 256.
#include <algorithm>

#include "common.cuh"
#include "tcgen05_ptx.cuh"

#define BUMP(L) do { if ((L).launches) ++*(L).launches; } while (0)

namespace {

constexpr int HD = 64;               // head dim
constexpr int KB = 64;               // keys per online-softmax block

__device__ __forceinline__ void ldsm_x4(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void ldsm_x4_t(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2, uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float* c, const uint32_t* a, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
        "{%0, %1, %2, %3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float a, float b) {
    __nv_bfloat162 h = __floats2bfloat162_rn(a, b);
    return *reinterpret_cast<uint32_t*>(&h);
}

// grid (q_slices, frames*heads); block = warps*32; dynamic smem = 2 * tpad * 128 bytes
__global__ void __launch_bounds__(512) attention_mma_kernel(const bf16* __restrict__ qkv, bf16* __restrict__ out,
                                                            int tokens, int heads, int tpad, int rows_per_cta) {
    extern __shared__ __align__(128) uint8_t smem[];
    const int f = blockIdx.y / heads, h = blockIdx.y % heads;
    const int d = heads * HD;
    const size_t row0 = (size_t)f * tokens;
    const bf16* base = qkv + row0 * 3 * d + h * HD;
    uint8_t* Ks = smem;
    uint8_t* Vs = smem + (size_t)tpad * 128;
    // ---- stage K and V: chunk c of row r lives at r*128 + ((c ^ (r & 7)) * 16); rows >= tokens are 0
    for (int i = threadIdx.x; i < tpad * 16; i += blockDim.x) {
        const int r = i >> 4, c = i & 7, isv = (i >> 3) & 1;
        uint4 v = make_uint4(0, 0, 0, 0);
        if (r < tokens) v = *reinterpret_cast<const uint4*>(base + (size_t)r * 3 * d + (1 + isv) * d + c * 8);
        *reinterpret_cast<uint4*>((isv ? Vs : Ks) + r * 128 + ((c ^ (r & 7)) << 4)) = v;
    }
    __syncthreads();

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int g = lane >> 2, t = lane & 3;
    const int q0 = blockIdx.x * rows_per_cta + warp * 16;
    if (q0 >= tokens) return;
    // ---- Q fragments (A operand), straight from global memory
    uint32_t qa[4][4];
    {
        const int r_lo = q0 + g, r_hi = q0 + g + 8;
#pragma unroll
        for (int ks = 0; ks < 4; ++ks) {
            const int c = ks * 16 + 2 * t;
            qa[ks][0] = r_lo < tokens ? *reinterpret_cast<const uint32_t*>(base + (size_t)r_lo * 3 * d + c) : 0u;
            qa[ks][1] = r_hi < tokens ? *reinterpret_cast<const uint32_t*>(base + (size_t)r_hi * 3 * d + c) : 0u;
            qa[ks][2] = r_lo < tokens ? *reinterpret_cast<const uint32_t*>(base + (size_t)r_lo * 3 * d + c + 8) : 0u;
            qa[ks][3] = r_hi < tokens ? *reinterpret_cast<const uint32_t*>(base + (size_t)r_hi * 3 * d + c + 8) : 0u;
        }
    }
    const uint32_t ks_addr = (uint32_t)__cvta_generic_to_shared(Ks);
    const uint32_t vs_addr = (uint32_t)__cvta_generic_to_shared(Vs);
    const float sl2 = 0.125f * 1.4426950408889634f;       // 1/sqrt(64) * log2(e)
    float o[8][4];
#pragma unroll
    for (int i = 0; i < 8; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
    float m_lo = -INFINITY, m_hi = -INFINITY, l_lo = 0.f, l_hi = 0.f;

    for (int k0 = 0; k0 < tokens; k0 += KB) {
        const int valid = min(KB, tokens - k0);
        const int nt16 = (valid + 15) >> 4;            // 16-key groups in this block
        float s[8][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) { s[i][0] = s[i][1] = s[i][2] = s[i][3] = 0.f; }
        // S = Q K^T
#pragma unroll
        for (int j = 0; j < 4; ++j) {                  // pairs of 8-key tiles
            if (j < nt16) {
#pragma unroll
                for (int ks = 0; ks < 4; ++ks) {
                    const int mi = lane >> 3;
                    const int r = k0 + j * 16 + (mi >> 1) * 8 + (lane & 7);
                    const int c = ks * 2 + (mi & 1);
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4(ks_addr + r * 128 + ((c ^ (r & 7)) << 4), b0, b1, b2, b3);
                    mma_bf16(s[2 * j], qa[ks], b0, b1);
                    mma_bf16(s[2 * j + 1], qa[ks], b2, b3);
                }
            }
        }
        // scale, mask, online softmax
        float bm_lo = -INFINITY, bm_hi = -INFINITY;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const int key = k0 + i * 8 + 2 * t;
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const bool ok = (key + (e & 1)) < tokens && (i >> 1) < nt16;
                s[i][e] = ok ? s[i][e] * sl2 : -INFINITY;
            }
            bm_lo = fmaxf(bm_lo, fmaxf(s[i][0], s[i][1]));
            bm_hi = fmaxf(bm_hi, fmaxf(s[i][2], s[i][3]));
        }
        bm_lo = fmaxf(bm_lo, __shfl_xor_sync(0xFFFFFFFFu, bm_lo, 1));
        bm_lo = fmaxf(bm_lo, __shfl_xor_sync(0xFFFFFFFFu, bm_lo, 2));
        bm_hi = fmaxf(bm_hi, __shfl_xor_sync(0xFFFFFFFFu, bm_hi, 1));
        bm_hi = fmaxf(bm_hi, __shfl_xor_sync(0xFFFFFFFFu, bm_hi, 2));
        const float nm_lo = fmaxf(m_lo, bm_lo), nm_hi = fmaxf(m_hi, bm_hi);   // finite: key k0 is valid
        const float cf_lo = exp2f(m_lo - nm_lo), cf_hi = exp2f(m_hi - nm_hi);
        m_lo = nm_lo; m_hi = nm_hi;
        float rs_lo = 0.f, rs_hi = 0.f;
        uint32_t pa[4][4];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float p0 = exp2f(s[i][0] - nm_lo), p1 = exp2f(s[i][1] - nm_lo);
            const float p2 = exp2f(s[i][2] - nm_hi), p3 = exp2f(s[i][3] - nm_hi);
            rs_lo += p0 + p1;
            rs_hi += p2 + p3;
            pa[i >> 1][(i & 1) * 2 + 0] = pack2(p0, p1);
            pa[i >> 1][(i & 1) * 2 + 1] = pack2(p2, p3);
        }
        l_lo = l_lo * cf_lo + rs_lo;
        l_hi = l_hi * cf_hi + rs_hi;
#pragma unroll
        for (int i = 0; i < 8; ++i) { o[i][0] *= cf_lo; o[i][1] *= cf_lo; o[i][2] *= cf_hi; o[i][3] *= cf_hi; }
        // O += P V
#pragma unroll
        for (int kk = 0; kk < 4; ++kk) {               // 16-key steps
            if (kk < nt16) {
#pragma unroll
                for (int n = 0; n < 4; ++n) {          // pairs of 8-dim tiles
                    const int mi = lane >> 3;
                    const int r = k0 + kk * 16 + (mi & 1) * 8 + (lane & 7);
                    const int c = n * 2 + (mi >> 1);
                    uint32_t b0, b1, b2, b3;
                    ldsm_x4_t(vs_addr + r * 128 + ((c ^ (r & 7)) << 4), b0, b1, b2, b3);
                    mma_bf16(o[2 * n], pa[kk], b0, b1);
                    mma_bf16(o[2 * n + 1], pa[kk], b2, b3);
                }
            }
        }
    }
    // row sums live in the 4 threads of a quad
    l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 1);
    l_lo += __shfl_xor_sync(0xFFFFFFFFu, l_lo, 2);
    l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 1);
    l_hi += __shfl_xor_sync(0xFFFFFFFFu, l_hi, 2);
    const float inv_lo = 1.f / l_lo, inv_hi = 1.f / l_hi;
    const int r_lo = q0 + g, r_hi = q0 + g + 8;
    bf16* obase = out + row0 * d + h * HD;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
        const int c = i * 8 + 2 * t;
        if (r_lo < tokens) *reinterpret_cast<uint32_t*>(obase + (size_t)r_lo * d + c) = pack2(o[i][0] * inv_lo, o[i][1] * inv_lo);
        if (r_hi < tokens) *reinterpret_cast<uint32_t*>(obase + (size_t)r_hi * d + c) = pack2(o[i][2] * inv_hi, o[i][3] * inv_hi);
    }
}
// ---------------------------------------------------------------------------------------
// tcgen05 attention.  One CTA per (frame, head); K and V of the head are brought in once by TMA
// (128B swizzle), the query rows are taken 128 at a time:
//     S = Q K^T            UMMA 128 x nb x 16, four K steps, fp32 scores in tensor memory
//     P = exp2(c (S - m))  four warps, one score row per thread (tcgen05.ld), written back over S
//                          as packed bf16 (tcgen05.st), row sums kept in registers
//     O = P V              UMMA 128 x 64 x 16 with the A operand read from tensor memory and V as
//                          an MN-major shared-memory operand, one K step per 16 keys
//     out = O / rowsum     tcgen05.ld, bf16, straight to global memory
// Keys come in blocks of up to 208 (13 x 16).  With one block (up to 208 tokens) the row maximum
// comes from the same scores.  With several blocks the scores are formed twice: a first sweep
// yields each row's maximum over all keys, the second forms P against that final maximum and
// accumulates O over the blocks, so no rescaling of O is ever needed.
// Tensor memory holds two regions of scores (208 columns each) and O behind them; the issuing thread
// forms the scores of the next step in the other region while the softmax warps sweep this one
// (per region: one mbarrier "scores formed", one "scores consumed"), and issues a block's P V
// product as soon as its probabilities are written.  ATT_SHARES softmax warps per lane quarter
// split the key columns of a block; they exchange row maxima and row sums through shared memory.
// (One key block goes to the pipelined kernel further down.)
// ---------------------------------------------------------------------------------------
constexpr int AQ = 128;                    // query rows per tile
constexpr int AKB = 208;                   // keys per score block
constexpr int ATT_MAX_SHARES = 3;          // softmax warps per lane quarter (they split the key columns)
#ifndef PM_ATT_SHARES
#define PM_ATT_SHARES 2
#endif
constexpr int ATT_SHARES = PM_ATT_SHARES;  // the multi-block kernel's choice: block = 32 + 128 * ATT_SHARES threads
constexpr int AQ_BYTES = AQ * 128;
constexpr int AKB_BYTES = AKB * 128;
constexpr int ATT_MAX_BLOCKS = 3;

struct AttnArgs {
    int tokens, heads, tpad, n_blocks, n_qtiles;
    int q_split;               // CTAs per (frame, head); each takes a contiguous share of the query tiles
    uint32_t tmem_cols, o_col;
    bf16* out;
    int* status;
};

// maximum of the first `lim` of 32 score columns (all of them if lim >= 32)
template <int N, bool MASK>
__device__ __forceinline__ float chunk_max(const uint32_t* v, int lim, float m) {
    float t[4] = {m, -INFINITY, -INFINITY, -INFINITY};       // four independent chains
#pragma unroll
    for (int j = 0; j < N; ++j) {
        const float sj = __uint_as_float(v[j]);
        t[j & 3] = fmaxf(t[j & 3], (!MASK || j < lim) ? sj : -INFINITY);
    }
    return fmaxf(fmaxf(t[0], t[1]), fmaxf(t[2], t[3]));
}
__device__ __forceinline__ float ex2_approx(float x) {     // one MUFU instruction; flushes denormals
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}
// p_j = exp2(c s_j - mc) (0 beyond lim), packed to bf16 pairs; returns the sum of the p_j
template <int N, bool MASK>
__device__ __forceinline__ float chunk_probs(const uint32_t* v, int lim, float c, float mc, uint32_t* packed) {
    float sum[4] = {0.f, 0.f, 0.f, 0.f};                     // four independent chains
#pragma unroll
    for (int j = 0; j < N; j += 2) {
        float p0 = ex2_approx(fmaf(__uint_as_float(v[j]), c, -mc));
        float p1 = ex2_approx(fmaf(__uint_as_float(v[j + 1]), c, -mc));
        if (MASK) { p0 = j < lim ? p0 : 0.f; p1 = j + 1 < lim ? p1 : 0.f; }
        sum[(j >> 1) & 3] += p0 + p1;
        packed[j >> 1] = pack2(p0, p1);
    }
    return (sum[0] + sum[1]) + (sum[2] + sum[3]);
}

// Sweep over the score columns [0, ncols) that start at tensor-memory address t_s (ncols a multiple
// of 16, `valid` of them real), 16 at a time with the next load in flight.  PROBS = false: running
// row maximum.  PROBS = true: P (packed bf16, 8 columns per 16 scores) goes to t_p onwards and the
// row sum of this range is added to acc.
template <bool PROBS>
__device__ __forceinline__ float score_range_sweep(uint32_t t_s, uint32_t t_p, int ncols, int valid, float c, float mc,
                                                   float acc) {
    uint32_t va[16], vb[16];
    auto piece = [&](const uint32_t* v, int c0) {
        const int lim = valid - c0;
        if (PROBS) {
            uint32_t pk[8];
            acc += lim >= 16 ? chunk_probs<16, false>(v, 16, c, mc, pk) : chunk_probs<16, true>(v, lim, c, mc, pk);
            tmem_st8(t_p + (uint32_t)(c0 >> 1), pk);
        } else {
            acc = lim >= 16 ? chunk_max<16, false>(v, 16, acc) : chunk_max<16, true>(v, lim, acc);
        }
    };
    tmem_ld16(t_s, va);
    tmem_ld_wait();
#pragma unroll 1
    for (int c0 = 0; c0 < ncols; c0 += 32) {
        if (c0 + 16 < ncols) tmem_ld16(t_s + (uint32_t)(c0 + 16), vb);
        piece(va, c0);
        tmem_ld_wait();
        if (c0 + 16 < ncols) {
            if (c0 + 32 < ncols) tmem_ld16(t_s + (uint32_t)(c0 + 32), va);
            piece(vb, c0 + 16);
            tmem_ld_wait();
        }
    }
    return acc;
}

// Share k of `shares` takes the 16-key pieces [att_first(shares, k), att_first(shares, k + 1)) of a key
// block (capped to the block's pieces) and leaves its P at the start of its own score columns.
__host__ __device__ constexpr int att_first(int shares, int k) {
    return shares == 1 ? (k == 0 ? 0 : 13) : shares == 2 ? (k == 0 ? 0 : k == 1 ? 7 : 13)
                                                         : (k == 0 ? 0 : k == 1 ? 5 : k == 2 ? 9 : 13);
}

template <int SHARES>
__global__ void __launch_bounds__(32 + 128 * SHARES, 1)
attention_tc_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kv,
                    const AttnArgs args) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if (base & 1023u) {                       // swizzled operands need a 1024-byte aligned window
        if (threadIdx.x == 0) atomicCAS(args.status, 0, (int)PM_ERR_CUDA);
        return;
    }
    const int fh = blockIdx.x / args.q_split, part = blockIdx.x % args.q_split;
    const int f = fh / args.heads, h = fh % args.heads;
    const int per = (args.n_qtiles + args.q_split - 1) / args.q_split;
    const int qt0 = part * per, qt1 = min(args.n_qtiles, qt0 + per);          // this CTA's query tiles
    const int d = args.heads * HD;
    const int T = args.tokens;
    const int n_blocks = args.n_blocks;
    const uint32_t q_s = base;
    const uint32_t k_s = q_s + AQ_BYTES;
    const uint32_t v_s = k_s + n_blocks * AKB_BYTES;
    const uint32_t bars = v_s + n_blocks * AKB_BYTES;
    // barriers: operands landed (kv, q); scores of a step formed, per score region (s_bar[2]); a step's scores
    // consumed by all softmax warps -- maxima taken, or probabilities written (c_bar[2]); O complete (o_bar);
    // O read out (ofree_bar); the shares' row maxima / row sums exchanged (max_bar, sum_bar)
    const uint32_t q_bar = bars + 8, o_bar = bars + 48, ofree_bar = bars + 56;
    auto k_bar = [&](int b) { return bars + 96u + 8u * (uint32_t)b; };       // key block b landed
    auto v_bar = [&](int b) { return bars + 120u + 8u * (uint32_t)b; };      // value block b landed
    const uint32_t max_bar = bars + 64, sum_bar = bars + 72;
    auto s_bar = [&](uint32_t r) { return bars + 16u + 8u * r; };
    auto c_bar = [&](uint32_t r) { return bars + 32u + 8u * r; };
    uint8_t* bar_ptr = smem_raw + (bars - base);
    float* xchg = reinterpret_cast<float*>(bar_ptr + 160);       // [max | sum][share][row]
    constexpr int shares = SHARES;
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_ptr + 80);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + 88);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // score steps of one query tile: with several key blocks the scores are formed twice (all of a row's
    // maxima must be known before its first exponential, and tensor memory holds two blocks of scores
    // beside O, not three): steps 0 .. n_blocks-1 for the maxima, n_blocks .. 2 n_blocks-1 for the
    // probabilities.  Step s of the CTA (all tiles) uses score region s % 2.
    const int n_steps = n_blocks > 1 ? 2 * n_blocks : 1;

    if (threadIdx.x == 0) {
        mbar_init(q_bar, 1);
        for (int b = 0; b < ATT_MAX_BLOCKS; ++b) { mbar_init(k_bar(b), 1); mbar_init(v_bar(b), 1); }
        for (uint32_t r = 0; r < 2; ++r) { mbar_init(s_bar(r), 1); mbar_init(c_bar(r), 4 * shares); }
        mbar_init(o_bar, 1); mbar_init(ofree_bar, 4 * shares);
        mbar_init(max_bar, 4 * shares); mbar_init(sum_bar, 4 * shares);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        // all operand loads of the head go out before tensor memory is requested, in the order of their
        // first use and each block on a barrier of its own: the first scores need the query tile and the
        // first key block only
        mbar_expect_tx(q_bar, AQ_BYTES);
        tma_load_2d(q_s, &tm_q, h * HD, f * T + qt0 * AQ, q_bar);
        for (int b = 0; b < n_blocks; ++b) {
            mbar_expect_tx(k_bar(b), (uint32_t)AKB_BYTES);
            tma_load_2d(k_s + b * AKB_BYTES, &tm_kv, d + h * HD, f * T + b * AKB, k_bar(b));
        }
        for (int b = 0; b < n_blocks; ++b) {
            mbar_expect_tx(v_bar(b), (uint32_t)AKB_BYTES);
            tma_load_2d(v_s + b * AKB_BYTES, &tm_kv, 2 * d + h * HD, f * T + b * AKB, v_bar(b));
        }
    }
    __syncwarp();
    if (warp == 0) {
        tmem_alloc(smem_u32((const void*)tmem_slot), args.tmem_cols);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const uint32_t o_tmem = tmem_base + args.o_col;

    if (warp == 0) {
        if (lane == 0) {
            // ------------------------------------------------------ TMA + MMA issue
            // The scores of step s + 1 are formed in the other region while the softmax warps are at step s;
            // products issued by this thread run in issue order, so a region's P V product is through
            // before the scores that are issued after it overwrite the region.
            const uint32_t idesc_pv = instr_desc_b_mn(HD);
            // descriptors built once; a K step adds 2 (32 B) for Q / K and 128 (2048 B) for V
            const uint64_t dq0 = smem_desc(q_s, 128), dk0 = smem_desc(k_s, 128), dv0 = smem_desc(v_s, 128);
            uint32_t s = 0;                                      // score steps issued so far
            bool ok = true;
            auto issue_scores = [&](int i) {                     // step i of the tile: key block i % n_blocks
                const int b = i % n_blocks;
                const uint32_t r = s & 1u;
                // the region's previous scores (step s - 2) must have been consumed
                ok = mbar_wait(c_bar(r), ((s >> 1) & 1u) ^ 1u, abort_flag, args.status);
                if (ok && s < (uint32_t)n_blocks) ok = mbar_wait(k_bar(b), 0, abort_flag, args.status);   // a block's first use
                if (!ok) return;
                tc_fence_after();
                const int nb = min(AKB, args.tpad - b * AKB);
                const uint32_t idesc_s = instr_desc(nb);
                const uint64_t bo = (uint64_t)((b * AKB_BYTES) >> 4);
#pragma unroll
                for (int k = 0; k < HD / 16; ++k)
                    umma_bf16(tmem_base + r * (uint32_t)AKB, dq0 + 2 * k, dk0 + bo + 2 * k, idesc_s, k > 0);
                umma_commit(s_bar(r));
                ++s;
            };
            for (int qt = qt0; qt < qt1 && ok; ++qt) {
                ok = mbar_wait(q_bar, (qt - qt0) & 1, abort_flag, args.status);
                if (!ok) break;
                tc_fence_after();
                const uint32_t s0 = s;                           // the tile's first step
                issue_scores(0);
                for (int i = 0; i < n_steps && ok; ++i) {
                    if (i + 1 < n_steps) issue_scores(i + 1);
                    if (!ok) break;
                    if (n_blocks > 1 && i < n_blocks) continue;  // a step for the maxima: nothing to multiply
                    const int b = i % n_blocks;
                    const uint32_t si = s0 + (uint32_t)i, r = si & 1u;
                    // the step's probabilities are written (so its scores, the tile's last ones included, exist)
                    ok = mbar_wait(c_bar(r), (si >> 1) & 1u, abort_flag, args.status);
                    if (ok && qt == qt0) ok = mbar_wait(v_bar(b), 0, abort_flag, args.status);          // a block's first use
                    if (!ok) break;
                    tc_fence_after();
                    if (b == n_blocks - 1 && qt + 1 < qt1) {
                        // the query rows are no longer needed: fetch the next tile's behind the P V products
                        mbar_expect_tx(q_bar, AQ_BYTES);
                        tma_load_2d(q_s, &tm_q, h * HD, f * T + (qt + 1) * AQ, q_bar);
                    }
                    if (b == 0 && qt > qt0) {
                        // the first product of a tile overwrites O: the previous tile's must have been read out
                        ok = mbar_wait(ofree_bar, (uint32_t)(qt - qt0 - 1) & 1u, abort_flag, args.status);
                        if (!ok) break;
                        tc_fence_after();
                    }
                    const int nb = min(AKB, args.tpad - b * AKB);
                    const uint64_t bo = (uint64_t)((b * AKB_BYTES) >> 4);
                    // P of piece kk sits where its share left it: at the start of that share's columns
                    uint32_t p_col = 0;
                    for (int kk = 0; kk < nb / 16; ++kk) {
                        if (kk == att_first(shares, 1) || kk == att_first(shares, 2)) p_col = (uint32_t)(kk * 16);
                        umma_bf16_ts(o_tmem, tmem_base + r * (uint32_t)AKB + p_col, dv0 + bo + 128 * kk, idesc_pv,
                                     (b > 0 || kk > 0) ? 1u : 0u);
                        p_col += 8;
                    }
                    if (b == n_blocks - 1) umma_commit(o_bar);
                }
            }
        }
    } else {
        // ---------------------------------------------------------- softmax + output
        const int quarter = warp & 3;                            // TMEM lanes 32*quarter .. +31
        const int share = (warp - 1) >> 2;                       // which share of the key columns
        const int row = quarter * 32 + lane;
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16);
        const float c = 0.125f * 1.4426950408889634f;            // 1/sqrt(64) * log2(e)
        float* maxes = xchg;                                     // [share][row]
        float* sums = xchg + ATT_MAX_SHARES * AQ;
        uint32_t s = 0, tile_no = 0;
        bool ok = true;
        // this warp's columns of key block b: [col0, col0 + ncols), `valid` of them real
        auto my_cols = [&](int b, int& col0, int& ncols, int& valid) {
            const int np = min(AKB, args.tpad - b * AKB) / 16;
            const int p0 = min(att_first(shares, share), np), p1 = min(att_first(shares, share + 1), np);
            col0 = p0 * 16; ncols = (p1 - p0) * 16; valid = T - b * AKB - col0;
        };
        for (int qt = qt0; qt < qt1 && ok; ++qt, ++tile_no) {
            const int q_row = qt * AQ + row;
            const bool warp_active = qt * AQ + quarter * 32 < T;      // else: no row of this warp exists
            float m = -INFINITY, l = 0.f;
            int col0, ncols, valid;
            for (int i = 0; i < n_steps; ++i, ++s) {
                const int b = i % n_blocks;
                const bool probs = n_blocks == 1 || i >= n_blocks;
                const uint32_t r = s & 1u;
                ok = mbar_wait(s_bar(r), (s >> 1) & 1u, abort_flag, args.status);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                tc_fence_after();
                const uint32_t t_s = t_lane + r * (uint32_t)AKB;
                my_cols(b, col0, ncols, valid);
                if (!probs || n_blocks == 1) {
                    if (warp_active && ncols > 0)
                        m = score_range_sweep<false>(t_s + (uint32_t)col0, 0u, ncols, valid, 0.f, 0.f, m);
                }
                if (probs) {
                    if (b == 0 && shares > 1) {
                        // the row maximum over all keys: every share's part, through shared memory
                        maxes[share * AQ + row] = m;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(max_bar);
                        ok = mbar_wait(max_bar, tile_no & 1u, abort_flag, args.status);
                        ok = __all_sync(0xFFFFFFFFu, ok);
                        if (!ok) break;
#pragma unroll
                        for (int k = 0; k < shares; ++k) m = fmaxf(m, maxes[k * AQ + row]);
                    }
                    if (warp_active && ncols > 0) {
                        l = score_range_sweep<true>(t_s + (uint32_t)col0, t_s + (uint32_t)col0, ncols, valid, c, m * c, l);
                        tmem_st_wait();
                    }
                    if (shares > 1 && b == n_blocks - 1) {
                        sums[share * AQ + row] = l;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(sum_bar);
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(c_bar(r));
            }
            if (!ok) break;
            if (shares > 1) {
                ok = mbar_wait(sum_bar, tile_no & 1u, abort_flag, args.status);
                ok = __all_sync(0xFFFFFFFFu, ok);
                if (!ok) break;
                l = 0.f;
#pragma unroll
                for (int k = 0; k < shares; ++k) l += sums[k * AQ + row];
            }
            // O = sum over the key blocks of P V is complete: the finished rows are written out
            ok = mbar_wait(o_bar, tile_no & 1u, abort_flag, args.status);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            {
                // the output columns are split between the first two shares (all 64 to the only one)
                const int ocols = shares == 1 ? 64 : 32;
                if (warp_active && share * ocols < 64) {
                    const float inv = 1.f / l;
                    bf16* orow = args.out + ((size_t)f * T + q_row) * d + h * HD + share * ocols;
                    for (int part = 0; part < ocols / 32; ++part) {
                        uint32_t v[32];
                        tmem_ld32((t_lane + args.o_col) + (uint32_t)(share * ocols + part * 32), v);
                        tmem_ld_wait();
                        if (q_row < T) {
                            // 32-byte stores: one full sector per row per instruction
#pragma unroll
                            for (int q = 0; q < 2; ++q) {
                                uint32_t o[8];
#pragma unroll
                                for (int e = 0; e < 8; ++e)
                                    o[e] = pack2(__uint_as_float(v[q * 16 + 2 * e]) * inv,
                                                 __uint_as_float(v[q * 16 + 2 * e + 1]) * inv);
                                asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                             ::"l"(orow + part * 32 + q * 16), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]),
                                               "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                                             : "memory");
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(ofree_bar);
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);    // let copies / MMAs in flight land
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 0) {
        tc_fence_after();
        tmem_dealloc(tmem_base, args.tmem_cols);
    }
}

// ---------------------------------------------------------------------------------------
// Pipelined variant for sequences of one key block (up to 208 tokens, at most two query tiles):
// one persistent CTA per SM walks (frame, head) items and keeps two query tiles in flight, each in
// its own half of tensor memory with its own group of eight softmax warps:
//     warp 0         TMA: K, V and the query tiles of item j+2 land while items j, j+1 are computed
//     warp 1         MMA issue:  S(c), then P V of tile c-1, then S(c+1), ...
//     warps 2..9     softmax + output of the even tiles (tensor-memory columns 0..255)
//     warps 10..17   the same for the odd tiles (columns 256..511)
// so the tensor pipe, the two softmax groups and the loads of the following items overlap inside one
// CTA.  Two warps share each quarter of the 128 rows (a warp reaches the tensor-memory lanes
// 32 (w mod 4) .. +31 only) and split the key columns: the first seven 16-key pieces and the rest.
// The sweeps are chains of dependent operations, so what bounds them is how many warps a scheduler
// can switch between: four per scheduler here against two with one warp per quarter.  The halves
// exchange their row maxima and row sums through shared memory (mbarriers, bounded waits).
// Column map of a tile's 256-column slot: scores 0..207; P of the first half over 0..55, P of the
// second half in 208..255 (so that it never lands on scores the first half still reads); O in
// 128..191 once both halves are done.  Tile c of a CTA is query tile c % nq of its item c / nq.
// ---------------------------------------------------------------------------------------
constexpr int APIPE_GROUP_WARPS = 8;
constexpr int APIPE_THREADS = 64 + 2 * 32 * APIPE_GROUP_WARPS;      // 576
constexpr int APIPE_ITEM_BYTES = 2 * AKB_BYTES + 2 * AQ_BYTES;      // K, V, two query tiles
constexpr int APIPE_SPLIT = 7;                                       // 16-key pieces of the first half
constexpr int APIPE_XCHG_BYTES = 2 * 2 * 2 * AQ * 4;                 // [max | sum][group][half][row]

struct AttnPipeArgs {
    int tokens, heads, tpad, nq, n_items;
    bf16* out;
    int* status;
};

__global__ void __launch_bounds__(APIPE_THREADS, 1)
attention_pipe_kernel(const __grid_constant__ CUtensorMap tm_q, const __grid_constant__ CUtensorMap tm_kv,
                      const AttnPipeArgs args) {
    extern __shared__ __align__(1024) uint8_t smem_raw[];
    const uint32_t base = smem_u32(smem_raw);
    if (base & 1023u) {                       // swizzled operands need a 1024-byte aligned window
        if (threadIdx.x == 0) atomicCAS(args.status, 0, (int)PM_ERR_CUDA);
        return;
    }
    const int T = args.tokens, nq = args.nq, d = args.heads * HD;
    const int my_items = (args.n_items - (int)blockIdx.x + (int)gridDim.x - 1) / (int)gridDim.x;
    const int my_tiles = my_items * nq;
    const int n_pieces = args.tpad / 16, split = min(APIPE_SPLIT, n_pieces);
    auto k_s = [&](int buf) { return base + buf * APIPE_ITEM_BYTES; };
    auto v_s = [&](int buf) { return base + buf * APIPE_ITEM_BYTES + AKB_BYTES; };
    auto q_s = [&](int buf, int qt) { return base + buf * APIPE_ITEM_BYTES + 2 * AKB_BYTES + qt * AQ_BYTES; };
    float* xchg = reinterpret_cast<float*>(smem_raw + 2 * APIPE_ITEM_BYTES);
    const uint32_t bars = base + 2 * APIPE_ITEM_BYTES + APIPE_XCHG_BYTES;
    auto kv_full = [&](int b) { return bars + 8u * b; };
    auto buf_free = [&](int b) { return bars + 16u + 8u * b; };
    auto s_ready = [&](int sl) { return bars + 32u + 8u * sl; };
    auto p_ready = [&](int sl) { return bars + 48u + 8u * sl; };
    auto o_ready = [&](int sl) { return bars + 64u + 8u * sl; };
    auto slot_free = [&](int sl) { return bars + 80u + 8u * sl; };
    auto max_bar = [&](int sl) { return bars + 96u + 8u * sl; };
    auto sum_bar = [&](int sl) { return bars + 112u + 8u * sl; };
    uint8_t* bar_ptr = smem_raw + (bars - base);
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(bar_ptr + 128);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(bar_ptr + 136);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int i = 0; i < 2; ++i) {
            mbar_init(kv_full(i), 1); mbar_init(buf_free(i), 1);
            mbar_init(s_ready(i), 1); mbar_init(p_ready(i), APIPE_GROUP_WARPS);
            mbar_init(o_ready(i), 1); mbar_init(slot_free(i), APIPE_GROUP_WARPS);
            mbar_init(max_bar(i), APIPE_GROUP_WARPS); mbar_init(sum_bar(i), APIPE_GROUP_WARPS);
        }
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == 1) {
        tmem_alloc(smem_u32((const void*)tmem_slot), 512);
        tmem_relinquish();
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;

    if (warp == 0) {
        if (lane == 0) {
            // ---------------------------------------------------------------- TMA producer
            bool ok = true;
            for (int j = 0; j < my_items && ok; ++j) {
                const int buf = j & 1;
                // the buffer's previous item (j - 2) must be through its last P V product
                ok = mbar_wait(buf_free(buf), (((uint32_t)j >> 1) & 1u) ^ 1u, abort_flag, args.status);
                if (!ok) break;
                const int item = (int)blockIdx.x + j * (int)gridDim.x;
                const int f = item / args.heads, h = item % args.heads;
                mbar_expect_tx(kv_full(buf), (uint32_t)(2 * AKB_BYTES + nq * AQ_BYTES));
                tma_load_2d(k_s(buf), &tm_kv, d + h * HD, f * T, kv_full(buf));
                for (int qt = 0; qt < nq; ++qt) tma_load_2d(q_s(buf, qt), &tm_q, h * HD, f * T + qt * AQ, kv_full(buf));
                tma_load_2d(v_s(buf), &tm_kv, 2 * d + h * HD, f * T, kv_full(buf));
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---------------------------------------------------------------- MMA issue
            const uint32_t idesc_s = instr_desc(args.tpad), idesc_pv = instr_desc_b_mn(HD);
            bool ok = true;
            // O(p) = P(p) V: P is the packed bf16 the two halves left in tile p's slot
            auto issue_pv = [&](int p) {
                const int slot = p & 1, buf = (p / nq) & 1;
                ok = mbar_wait(p_ready(slot), ((uint32_t)p >> 1) & 1u, abort_flag, args.status);
                if (!ok) return;
                tc_fence_after();
                const uint32_t s_tmem = tmem_base + (uint32_t)(slot * 256);
                const uint64_t dv0 = smem_desc(v_s(buf), 128);
                for (int kk = 0; kk < n_pieces; ++kk) {
                    const uint32_t p_col = kk < split ? (uint32_t)(kk * 8) : (uint32_t)(208 + (kk - split) * 8);
                    umma_bf16_ts(s_tmem + 128u, s_tmem + p_col, dv0 + 128 * kk, idesc_pv, kk > 0 ? 1u : 0u);
                }
                umma_commit(o_ready(slot));
                if (p % nq == nq - 1) umma_commit(buf_free(buf));     // the item's operands are no longer read
            };
            for (int c = 0; c < my_tiles && ok; ++c) {
                const int j = c / nq, qt = c % nq, buf = j & 1, slot = c & 1;
                if (qt == 0) ok = mbar_wait(kv_full(buf), ((uint32_t)j >> 1) & 1u, abort_flag, args.status);
                // the slot's previous tile (c - 2) must have been read out
                ok = ok && mbar_wait(slot_free(slot), (((uint32_t)c >> 1) & 1u) ^ 1u, abort_flag, args.status);
                if (!ok) break;
                tc_fence_after();
                const uint64_t dq0 = smem_desc(q_s(buf, qt), 128), dk0 = smem_desc(k_s(buf), 128);
#pragma unroll
                for (int k = 0; k < HD / 16; ++k)
                    umma_bf16(tmem_base + (uint32_t)(slot * 256), dq0 + 2 * k, dk0 + 2 * k, idesc_s, k > 0);
                umma_commit(s_ready(slot));
                if (c >= 1) issue_pv(c - 1);
            }
            if (ok && my_tiles > 0) issue_pv(my_tiles - 1);
        }
    } else {
        // -------------------------------------------------------------------- softmax + output
        const int group = (warp - 2) / APIPE_GROUP_WARPS;        // 0: even tiles, 1: odd tiles
        const int half = ((warp - 2) % APIPE_GROUP_WARPS) >> 2;  // which share of the key columns
        const int quarter = warp & 3;                            // TMEM lanes 32*quarter .. +31
        const int row = quarter * 32 + lane;                     // row of the query tile
        const uint32_t t_lane = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(group * 256);
        const int col0 = half == 0 ? 0 : split * 16;             // first key column of this warp
        const int ncols = half == 0 ? split * 16 : (n_pieces - split) * 16;
        const uint32_t t_p = t_lane + (half == 0 ? 0u : 208u);   // where this warp's P goes
        float* my_max = xchg + ((0 * 2 + group) * 2 + half) * AQ;
        float* other_max = xchg + ((0 * 2 + group) * 2 + (half ^ 1)) * AQ;
        float* my_sum = xchg + ((1 * 2 + group) * 2 + half) * AQ;
        float* other_sum = xchg + ((1 * 2 + group) * 2 + (half ^ 1)) * AQ;
        const float c_ = 0.125f * 1.4426950408889634f;           // 1/sqrt(64) * log2(e)
        bool ok = true;
        for (int c = group; c < my_tiles && ok; c += 2) {
            const uint32_t par = ((uint32_t)c >> 1) & 1u;
            const int j = c / nq, qt = c % nq;
            const int item = (int)blockIdx.x + j * (int)gridDim.x;
            const int f = item / args.heads, h = item % args.heads;
            const int q_row = qt * AQ + row;
            const bool warp_active = qt * AQ + quarter * 32 < T;     // else: no row of this warp exists
            ok = mbar_wait(s_ready(group), par, abort_flag, args.status);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            // row maximum: own columns, then the other half's through shared memory
            float m = -INFINITY;
            if (warp_active && ncols > 0)
                m = score_range_sweep<false>(t_lane + (uint32_t)col0, 0u, ncols, T - col0, 0.f, 0.f, m);
            my_max[row] = m;
            __syncwarp();
            if (lane == 0) mbar_arrive(max_bar(group));
            ok = mbar_wait(max_bar(group), par, abort_flag, args.status);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            m = fmaxf(m, other_max[row]);
            float l = 0.f;
            if (warp_active && ncols > 0) {
                l = score_range_sweep<true>(t_lane + (uint32_t)col0, t_p, ncols, T - col0, c_, m * c_, 0.f);
                tmem_st_wait();
            }
            my_sum[row] = l;
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { mbar_arrive(sum_bar(group)); mbar_arrive(p_ready(group)); }
            ok = mbar_wait(sum_bar(group), par, abort_flag, args.status);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            l += other_sum[row];
            ok = mbar_wait(o_ready(group), par, abort_flag, args.status);
            ok = __all_sync(0xFFFFFFFFu, ok);
            if (!ok) break;
            tc_fence_after();
            if (warp_active) {
                // each half writes 32 of the 64 output columns
                const float inv = 1.f / l;
                bf16* orow = args.out + ((size_t)f * T + q_row) * d + h * HD + half * 32;
                uint32_t v[32];
                tmem_ld32((t_lane + 128u) + (uint32_t)(half * 32), v);
                tmem_ld_wait();
                if (q_row < T) {
#pragma unroll
                    for (int q = 0; q < 2; ++q) {
                        uint32_t o[8];
#pragma unroll
                        for (int e = 0; e < 8; ++e)
                            o[e] = pack2(__uint_as_float(v[q * 16 + 2 * e]) * inv,
                                         __uint_as_float(v[q * 16 + 2 * e + 1]) * inv);
                        asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};"
                                     ::"l"(orow + q * 16), "r"(o[0]), "r"(o[1]), "r"(o[2]), "r"(o[3]),
                                       "r"(o[4]), "r"(o[5]), "r"(o[6]), "r"(o[7])
                                     : "memory");
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(slot_free(group));
        }
    }

    // ---------------------------------------------------------------------- teardown
    __syncwarp();
    if (*abort_flag) {
        for (int i = 0; i < 1000; ++i) __nanosleep(1000);    // let copies / MMAs in flight land
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, 512);
    }
}

}  // namespace

bool attention_tc_supported(int tokens) { return (tokens + 15) / 16 * 16 <= ATT_MAX_BLOCKS * AKB; }

bool attention_encode_maps(const bf16* qkv, int n_frames, int tokens, int heads, CUtensorMap* tm_q,
                           CUtensorMap* tm_kv) {
    const uint64_t w = (uint64_t)3 * heads * HD, rows = (uint64_t)n_frames * tokens;
    return tm_encode_2d(tm_q, qkv, w, rows, w * 2, HD, AQ, 128) &&
           tm_encode_2d(tm_kv, qkv, w, rows, w * 2, HD, AKB, 128);
}

cudaError_t launch_attention_tc(const Launch& L, const CUtensorMap& tm_q, const CUtensorMap& tm_kv,
                                bf16* out, int n_frames, int tokens, int heads, int n_sms) {
    if (n_frames <= 0) return cudaSuccess;
    AttnArgs a;
    a.tokens = tokens; a.heads = heads;
    a.tpad = (tokens + 15) / 16 * 16;
    a.n_blocks = (a.tpad + AKB - 1) / AKB;
    a.n_qtiles = (tokens + AQ - 1) / AQ;
    // one key block: a CTA per head (three fit an SM).  Several key blocks: one CTA per SM, so each
    // head's query tiles are spread over several CTAs when there are too few heads to fill the GPU.
    a.q_split = (a.n_blocks > 1 && n_frames * heads < 4 * 148) ? a.n_qtiles : 1;
    // two regions of scores (208 columns each), O behind them
    a.tmem_cols = 512u;
    a.o_col = 2u * AKB;
    a.out = out; a.status = L.status;
    if (a.n_blocks == 1 && a.n_qtiles <= 2 && n_sms > 0) {
        // one key block: the pipelined persistent kernel
        AttnPipeArgs pa;
        pa.tokens = tokens; pa.heads = heads; pa.tpad = a.tpad; pa.nq = a.n_qtiles;
        pa.n_items = n_frames * heads; pa.out = out; pa.status = L.status;
        const size_t psmem = 2 * (size_t)APIPE_ITEM_BYTES + APIPE_XCHG_BYTES + 192;
        static SmemGrant grant;
        if (cudaError_t e = grant.ensure(attention_pipe_kernel, (int)psmem); e != cudaSuccess) return e;
        ProfScope ps(L, KC_ATTENTION);
        attention_pipe_kernel<<<std::min(pa.n_items, n_sms), APIPE_THREADS, psmem, L.st>>>(tm_q, tm_kv, pa);
        BUMP(L);
        return cudaGetLastError();
    }
    // all of tensor memory and most of the shared memory: one CTA per SM
    size_t smem = (size_t)AQ_BYTES + (size_t)a.n_blocks * 2 * AKB_BYTES + 160 + 2 * ATT_MAX_SHARES * AQ * sizeof(float);
    static SmemGrant grant;
    if (cudaError_t e = grant.ensure(attention_tc_kernel<ATT_SHARES>, (int)smem); e != cudaSuccess) return e;
    ProfScope ps(L, KC_ATTENTION);
    attention_tc_kernel<ATT_SHARES><<<n_frames * heads * a.q_split, 32 + 128 * ATT_SHARES, smem, L.st>>>(tm_q, tm_kv, a);
    BUMP(L);
    return cudaGetLastError();
}

cudaError_t launch_attention_mma(const Launch& L, const bf16* qkv, bf16* out, int n_frames, int tokens,
                                 int heads) {
    if (n_frames <= 0) return cudaSuccess;
    const int groups = (tokens + 15) / 16;
    const int slices = (groups + 15) / 16;
    const int warps = (groups + slices - 1) / slices;
    const int tpad = groups * 16;
    const size_t smem = (size_t)tpad * 256;
    if (smem > 227 * 1024) return launch_attention_simple<bf16>(L, qkv, out, n_frames, tokens, heads);
    static SmemGrant grant;
    if (cudaError_t e = grant.ensure(attention_mma_kernel, (int)smem); e != cudaSuccess) return e;
    ProfScope ps(L, KC_ATTENTION);
    dim3 grid(slices, n_frames * heads);
    attention_mma_kernel<<<grid, warps * 32, smem, L.st>>>(qkv, out, tokens, heads, tpad, warps * 16);
    BUMP(L);
    return cudaGetLastError();
}
